// C ABI of the LAGA hot path (see include/laga.h): argument validation, TMA tensor-map
// construction, workspace carving and kernel launches on the caller's stream.
#include "../../include/laga.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <cstring>
#include <initializer_list>
#include <mutex>
#include <vector>

#include "attn_absorbed_sm100.cuh"
#include "attn_bwd_fused_sm100.cuh"
#include "attn_bwd_sm100.cuh"
#include "attn_fwd_sm100.cuh"
#include "gemm_sm100.cuh"
#include "layernorm_sm100.cuh"

namespace {

using namespace laga;

constexpr int kDc = 512, kDn = 128, kDr = 64, kDv = 128;
constexpr size_t kStatusBytes = 1024;   // the status word's slot; keeps what follows 1024-aligned

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The head geometry is fixed (the attention kernels' tiles and TMEM maps are built for it); the latent width
// is not: it only enters the three token-wise GEMMs, which take any multiple of 8 (16-byte rows).  The absorbed
// comparison form and the fused K/V rebuild are written for d_c = 512 (geometry_is_v3).
bool geometry_supported(int d_c, int d_nope, int d_rope, int d_v) {
    return d_c >= 8 && d_c <= 8192 && d_c % 8 == 0 && d_nope == kDn && d_rope == kDr && d_v == kDv;
}
bool geometry_is_v3(int d_c, int d_nope, int d_rope, int d_v) {
    return d_c == kDc && d_nope == kDn && d_rope == kDr && d_v == kDv;
}

// cuTensorMapEncodeTiled is resolved through the runtime so the library has no link-time
// dependency on the driver library (it must load on machines without a GPU).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor map, 128-byte swizzle, box of 64 contiguous elements x box_rows rows,
// out-of-range elements read as zero.
bool make_tmap_bf16(CUtensorMap* map, const void* base, uint64_t inner_elems, uint64_t rows,
                    uint64_t row_stride_bytes, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner_elems, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {64u, box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---- launch status slot ---------------------------------------------------------------------------
// The first kStatusBytes of every workspace: word 0 is the device status word; the work counters of the
// persistent attention kernels and their clock probes follow.  The first kStatusClearBytes (all of
// that) are cleared at the start of every entry point.
constexpr size_t kStatusClearBytes = 256;
constexpr size_t kCounterOffsetWords = 4;     // words 4, 5, 6: forward, dK/dV and dQ kernel work counters
constexpr size_t kProbeOffsetBytes = 64;      // four ClockProbe records (forward, dK/dV, dQ, fused backward)
enum { kSlotFwd = 0, kSlotDkv = 1, kSlotDq = 2, kSlotFused = 3 };
static_assert(kProbeOffsetBytes + 4 * sizeof(ClockProbe) <= kStatusClearBytes, "the probes must lie inside the cleared part of the slot");

unsigned* slot_counter(unsigned* status, int slot) { return status + kCounterOffsetWords + slot; }
ClockProbe* slot_probe(unsigned* status, int slot) {
    return reinterpret_cast<ClockProbe*>(reinterpret_cast<uint8_t*>(status) + kProbeOffsetBytes) + slot;
}

int launch_status() { return cudaGetLastError() == cudaSuccess ? LAGA_OK : LAGA_ERR_CUDA; }

// ---- per-device facts, looked up once per device (thread-safe) ------------------------------------
constexpr int kMaxDevices = 64;
constexpr int kGemmStages = 6;      // 64-deep k-stages of the CTA-pair GEMM (32 KB each)
struct DeviceInfo {
    std::once_flag once;
    int rc = LAGA_ERR_CUDA;
    int sms = 148;
    int fused_pairs = 74;               // CTA pairs of the fused backward that are resident at the same time
    std::once_flag scratch_once;
    unsigned char* builtin_scratch = nullptr;
};
DeviceInfo g_devices[kMaxDevices];

template <typename Kernel>
bool allow_smem(Kernel kernel, int bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

void init_device(DeviceInfo* info, int dev) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return;
    if (major != 10) { info->rc = LAGA_ERR_UNSUPPORTED; return; }
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) info->sms = sms;
    // every kernel of the library asks for more than the default 48 KB of dynamic shared memory: opt in once
    using G = GemmPairSmem<256, kGemmStages>;
    bool ok = allow_smem(gemm_pair_sm100_kernel<256, kGemmStages, false, true, EPI_BF16>, G::kTotalBytes) &&
              allow_smem(gemm_pair_sm100_kernel<256, kGemmStages, false, false, EPI_BF16>, G::kTotalBytes) &&
              allow_smem(gemm_pair_sm100_kernel<128, kGemmStages, false, false, EPI_BF16>, GemmPairSmem<128, kGemmStages>::kTotalBytes) &&
              allow_smem(gemm_pair_sm100_kernel<128, kGemmStages, false, true, EPI_BF16>, GemmPairSmem<128, kGemmStages>::kTotalBytes) &&
              allow_smem(gemm_pair_sm100_kernel<256, kGemmStages, true, true, EPI_ATOMIC_F32>, G::kTotalBytes) &&
              allow_smem(gemm_sm100_kernel<128, 4, false, true, EPI_BF16>, GemmSmem<128, 4>::kTotalBytes) &&
              allow_smem(attn_absorbed_fwd_sm100_kernel<true>, AttnAbsorbedSmem::kTotalBytes) &&
              allow_smem(attn_absorbed_fwd_sm100_kernel<false>, AttnAbsorbedSmem::kTotalBytes) &&
              allow_smem(attn_fwd_sm100_kernel<true>, AttnFwdSmem::kTotalBytes) &&
              allow_smem(attn_fwd_sm100_kernel<false>, AttnFwdSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dkv_sm100_kernel<true>, AttnBwdDkvSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dkv_sm100_kernel<false>, AttnBwdDkvSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dkv_sm100_kernel<true, true>, AttnBwdDkvSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dkv_sm100_kernel<false, true>, AttnBwdDkvSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dq_sm100_kernel<true>, AttnBwdDqSmem::kTotalBytes) &&
              allow_smem(attn_bwd_dq_sm100_kernel<false>, AttnBwdDqSmem::kTotalBytes) &&
              allow_smem(attn_bwd_fused_sm100_kernel<true>, AttnBwdFusedSmem::kTotalBytes) &&
              allow_smem(attn_bwd_fused_sm100_kernel<false>, AttnBwdFusedSmem::kTotalBytes);
    if (ok) {
        // The fused backward assigns work to pairs statically, so its grid must not exceed the pairs the
        // device keeps resident at once (SMs that cannot form a pair inside their GPC stay idle).
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(info->sms / 2 * 2), 1, 1);
        cfg.blockDim = dim3(kBwdThreads, 1, 1);
        cfg.dynamicSmemBytes = AttnBwdFusedSmem::kTotalBytes;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, attn_bwd_fused_sm100_kernel<true>, &cfg) == cudaSuccess && clusters > 0)
            info->fused_pairs = clusters < info->sms / 2 ? clusters : info->sms / 2;
        else {
            (void)cudaGetLastError();
            info->fused_pairs = info->sms / 2;
        }
    }
    info->rc = ok ? LAGA_OK : LAGA_ERR_CUDA;
    if (!ok) (void)cudaGetLastError();
}

// The current device's record; LAGA_ERR_UNSUPPORTED if it is not an sm_100 part.
int current_device(DeviceInfo** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LAGA_ERR_CUDA;
    DeviceInfo* info = &g_devices[dev];
    std::call_once(info->once, init_device, info, dev);
    *out = info;
    return info->rc;
}

int check_device() {
    DeviceInfo* info = nullptr;
    return current_device(&info);
}

int sm_count() {
    DeviceInfo* info = nullptr;
    return current_device(&info) == LAGA_OK ? info->sms : 148;
}

int fused_pair_count() {
    DeviceInfo* info = nullptr;
    return current_device(&info) == LAGA_OK ? info->fused_pairs : 74;
}

// Every data pointer must be device memory of the CURRENT device (or managed memory): a kernel given
// another device's pointer would fault, or silently use the wrong memory where peers are mapped.
int check_pointers(std::initializer_list<const void*> ptrs) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LAGA_ERR_CUDA;
    for (const void* p : ptrs) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
            (void)cudaGetLastError();
            return LAGA_ERR_INVALID_ARG;
        }
        if (attr.type == cudaMemoryTypeManaged) continue;
        if (attr.type != cudaMemoryTypeDevice || attr.device != dev) return LAGA_ERR_INVALID_ARG;
    }
    return LAGA_OK;
}

// Persistent kernels launch one CTA per SM (fewer if there are fewer tiles).
unsigned persistent_grid(int total_tiles) {
    const int sms = sm_count();
    return static_cast<unsigned>(total_tiles < sms ? (total_tiles < 1 ? 1 : total_tiles) : sms);
}

// The CTA-pair GEMM launches whole pairs: one pair per two SMs (fewer if there are fewer 256-row tiles).
unsigned pair_grid(int total_tiles) {
    const int pairs = sm_count() / 2;
    return 2u * static_cast<unsigned>(total_tiles < pairs ? (total_tiles < 1 ? 1 : total_tiles) : pairs);
}

// ---- tensor-map cache ------------------------------------------------------------------------------
// Encoding a tensor map is a driver call of a microsecond or two and an entry point needs up to five; for
// short sequences that is a visible part of the host time per call.  A map is a pure function of
// (base, extents, stride, box), so recently used ones are kept (64 entries, replaced round-robin).
struct TmapKey {
    const void* base;
    uint64_t inner, rows, stride;
    uint32_t box_rows;
    bool operator==(const TmapKey& o) const {
        return base == o.base && inner == o.inner && rows == o.rows && stride == o.stride && box_rows == o.box_rows;
    }
};
struct TmapCache {
    static constexpr int kEntries = 64;
    std::mutex mutex;
    TmapKey keys[kEntries] = {};
    CUtensorMap maps[kEntries];
    bool used[kEntries] = {};
    int next = 0;
};
TmapCache g_tmaps;

bool cached_tmap_bf16(CUtensorMap* map, const void* base, uint64_t inner_elems, uint64_t rows, uint64_t row_stride_bytes,
                      uint32_t box_rows) {
    const TmapKey key{base, inner_elems, rows, row_stride_bytes, box_rows};
    std::lock_guard<std::mutex> lock(g_tmaps.mutex);
    for (int i = 0; i < TmapCache::kEntries; ++i)
        if (g_tmaps.used[i] && g_tmaps.keys[i] == key) { *map = g_tmaps.maps[i]; return true; }
    if (!make_tmap_bf16(map, base, inner_elems, rows, row_stride_bytes, box_rows)) return false;
    const int slot = g_tmaps.next;
    g_tmaps.next = (slot + 1) % TmapCache::kEntries;
    g_tmaps.keys[slot] = key;
    g_tmaps.maps[slot] = *map;
    g_tmaps.used[slot] = true;
    return true;
}

// ---- launches ----------------------------------------------------------------------------------------
// Every kernel is launched through here.  `overlap` asks for programmatic dependent launch: the kernel may be
// scheduled while the kernel enqueued just before it on the stream is still running, and runs its set-up
// there; its threads then wait (griddepcontrol.wait, which every kernel of the library executes first thing
// after set-up) until that kernel has completed.  Only launches that directly follow another launch of the
// same entry point ask for it: the first kernel after a memset, a copy or the caller's own work is launched
// the ordinary way.
template <typename... Params, typename... Args>
void launch_kernel(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t stream, bool overlap,
                   Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = overlap ? &attr : nullptr;
    cfg.numAttrs = overlap ? 1 : 0;
    (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);   // the caller reads cudaGetLastError
}

// ---- measurement aid (laga_profile_kernel) ---------------------------------------------------------
// Caller-provided CUDA events recorded around launches of one kernel, cycling through the registered pairs.
struct ProfileSlot {
    std::vector<cudaEvent_t> starts, stops;
    unsigned long long launches = 0;
};
ProfileSlot g_profile[LAGA_KERNEL_COUNT];
std::mutex g_profile_mutex;

struct ScopedKernelEvents {
    cudaEvent_t stop = nullptr;
    cudaStream_t stream;
    ScopedKernelEvents(int kernel_id, cudaStream_t st) : stream(st) {
        std::lock_guard<std::mutex> lock(g_profile_mutex);
        ProfileSlot& slot = g_profile[kernel_id];
        if (!slot.starts.empty()) {
            const size_t i = static_cast<size_t>(slot.launches++ % slot.starts.size());
            cudaEventRecord(slot.starts[i], stream);
            stop = slot.stops[i];
        }
    }
    ~ScopedKernelEvents() {
        if (stop) cudaEventRecord(stop, stream);
    }
};

// How many of the h heads the persistent attention kernels sweep position by position instead of head by
// head (see work_sched.cuh): as many as keep the swept heads' streamed operands (640 bytes per token and
// head: K_nope, V and the rope band on one side, Q and dO on the other) within half of the 126 MB L2.
WorkSchedule make_schedule(int n_tiles, int S, int h, unsigned* counter, const int4* tiles = nullptr) {
    const long long per_head = static_cast<long long>(S) * 640;
    long long banded = (64ll << 20) / (per_head > 0 ? per_head : 1);
    if (banded < 1) banded = 1;
    if (banded > h) banded = h;
    return WorkSchedule{n_tiles, h, static_cast<int>(banded), n_tiles * h, counter, tiles};
}

// ---- y[M, N] = x[M, K] . W[K, N]: Algorithm 1 step 4 (KV = c_kv W, K = d_c) and the dense projections of
// ---- steps 1 and 7 through laga_linear --------------------------------------------------------------
template <int BN>
int launch_up_project_bn(const void* c_kv, const void* w, int S, int N, void* kv, unsigned* status,
                         cudaStream_t stream, bool overlap, int K) {
    constexpr int STAGES = kGemmStages;
    auto kernel = gemm_pair_sm100_kernel<BN, STAGES, false, true, EPI_BF16>;
    using L = GemmPairSmem<BN, STAGES>;
    CUtensorMap ta, tb;
    if (!cached_tmap_bf16(&ta, c_kv, K, S, static_cast<uint64_t>(K) * 2, 128)) return LAGA_ERR_CUDA;     // rows = tokens, inner = K
    if (!cached_tmap_bf16(&tb, w, N, K, static_cast<uint64_t>(N) * 2, 64)) return LAGA_ERR_CUDA;        // rows = K
    CUtensorMap tc;                                                                    // output boxes of 64 columns x 32 rows
    if (!cached_tmap_bf16(&tc, kv, N, S, static_cast<uint64_t>(N) * 2, 32)) return LAGA_ERR_CUDA;
    GemmArgs a{S, N, K, (K + 63) / 64, 1, kv, N, status, nullptr, 0, 1, 0, 0, 0};
    dim3 grid(pair_grid(((N + BN - 1) / BN) * ((S + 255) / 256)), 1, 1);
    { ScopedKernelEvents ev(LAGA_KERNEL_UP_PROJECT, stream); launch_kernel(kernel, grid, dim3(192), L::kTotalBytes, stream, overlap, ta, tb, tc, a); }
    return launch_status();
}
int launch_up_project(const void* c_kv, const void* w, int S, int N, void* kv, unsigned* status,
                      cudaStream_t stream, bool overlap = false, int K = kDc) {
    // As for dc_kv below: when 256-column tiles do not even give every CTA pair one tile, tiles of half the width
    // do better (S = 512, N = 512: 12.7 -> 10.7 us).  Where they only fill the LAST wave better they lose: at
    // S = 4096, N = 4096 (256 tiles on 74 pairs, four waves for 3.46) 26.8 us against 24.0.
    const int tiles_256 = ((N + 255) / 256) * ((S + 255) / 256);
    if (tiles_256 < sm_count() / 2) return launch_up_project_bn<128>(c_kv, w, S, N, kv, status, stream, overlap, K);
    return launch_up_project_bn<256>(c_kv, w, S, N, kv, status, stream, overlap, K);
}

// ---- Section 5.2, back through step 4 -----------------------------------------------------------
// dc_kv[S, d_c] = dKV[S, N] . W^T          (A = dKV K-major, B = W rows d_c / inner N: K-major)
// `clear` (optional) is an fp32 buffer of clear_floats elements this launch zeroes on its way in: the dW
// GEMM that follows accumulates into it with atomics.
template <int BN>
int launch_dckv_bn(const void* dkv, const void* w, int S, int N, void* dc_kv, float* clear, size_t clear_floats,
                   unsigned* status, cudaStream_t stream, bool overlap, int K) {
    constexpr int STAGES = kGemmStages;
    auto kernel = gemm_pair_sm100_kernel<BN, STAGES, false, false, EPI_BF16>;
    using L = GemmPairSmem<BN, STAGES>;
    CUtensorMap ta, tb;
    if (!cached_tmap_bf16(&ta, dkv, N, S, static_cast<uint64_t>(N) * 2, 128)) return LAGA_ERR_CUDA;
    if (!cached_tmap_bf16(&tb, w, N, K, static_cast<uint64_t>(N) * 2, BN / 2)) return LAGA_ERR_CUDA;
    CUtensorMap tc;
    if (!cached_tmap_bf16(&tc, dc_kv, K, S, static_cast<uint64_t>(K) * 2, 32)) return LAGA_ERR_CUDA;
    GemmArgs a{S, K, N, (N + 63) / 64, 1, dc_kv, K, status, reinterpret_cast<float4*>(clear), clear_floats / 4, 1, 0, 0, 0};
    dim3 grid(pair_grid(((K + BN - 1) / BN) * ((S + 255) / 256)), 1, 1);
    { ScopedKernelEvents ev(LAGA_KERNEL_DCKV_GEMM, stream); launch_kernel(kernel, grid, dim3(192), L::kTotalBytes, stream, overlap, ta, tb, tc, a); }
    return launch_status();
}
// (K: the width of the output, d_c for the path itself)
int launch_dckv(const void* dkv, const void* w, int S, int N, void* dc_kv, float* clear, size_t clear_floats,
                unsigned* status, cudaStream_t stream, bool overlap = false, int K = kDc) {
    // With 256-column tiles a short sequence leaves most CTA pairs without a tile when the output is narrow
    // (d_c = 512, S = 4096: 32 tiles for 74 pairs).  Narrower tiles double the count at the price of reading the
    // dKV rows once more from L2.
    const int tiles_256 = ((K + 255) / 256) * ((S + 255) / 256);
    if (tiles_256 < sm_count() / 2)
        return launch_dckv_bn<128>(dkv, w, S, N, dc_kv, clear, clear_floats, status, stream, overlap, K);
    return launch_dckv_bn<256>(dkv, w, S, N, dc_kv, clear, clear_floats, status, stream, overlap, K);
}

// dW[d_c, N] += c_kv^T . dKV   (both operands read with the token index as K: MN-major), split over
// the sequence with fp32 atomic accumulation into a buffer the caller of this function has cleared
// (launch_dckv does it) or wants added to.
int launch_dw(const void* c_kv, const void* dkv, int S, int N, float* dw, bool deterministic,
              unsigned* status, cudaStream_t stream, bool overlap = false, int K = kDc) {
    constexpr int BN = 256, STAGES = kGemmStages;
    auto kernel = gemm_pair_sm100_kernel<BN, STAGES, true, true, EPI_ATOMIC_F32>;
    using L = GemmPairSmem<BN, STAGES>;
    CUtensorMap ta, tb;
    if (!cached_tmap_bf16(&ta, c_kv, K, S, static_cast<uint64_t>(K) * 2, 64)) return LAGA_ERR_CUDA;
    if (!cached_tmap_bf16(&tb, dkv, N, S, static_cast<uint64_t>(N) * 2, 64)) return LAGA_ERR_CUDA;
    // Split the sequence to fill the persistent grid, but every split adds one fp32 atomic pass over the whole
    // [K, N] output.  Measured on B200: the atomics of one pass move at about 4.2 TB/s and the tiles run at
    // about 1.3 PFLOP/s times the fill of the last wave, so pick the split count that minimises
    //     flops / (1.3e15 * fill(s)) + s * output bytes / 4.2e12
    // (S = 4096, h = 16: 2 splits, 25 us, where filling the grid to 97 % with 9 splits took 39 us).
    const int tiles = ((K + 255) / 256) * ((N + BN - 1) / BN);
    const int k_tiles = (S + 63) / 64;
    const int sms = sm_count() / 2;       // CTA pairs
    int splits = 1;
    double best = 1e30;
    const double flops = 2.0 * S * K * N, out_bytes = static_cast<double>(K) * N * sizeof(float);
    for (int s = 1; s <= 16 && s <= k_tiles && !deterministic; ++s) {   // one split: one add per element
        const int total = tiles * s;
        const double fill = static_cast<double>(total) / (static_cast<double>((total + sms - 1) / sms) * sms);
        const double cost = flops / (1.3e15 * fill) + s * out_bytes / 4.2e12;
        if (cost < best) { best = cost; splits = s; }
    }
    const int per_split = (k_tiles + splits - 1) / splits;
    splits = (k_tiles + per_split - 1) / per_split;
    GemmArgs a{K, N, S, per_split, splits, dw, N, status, nullptr, 0, 1, 0, 0, 0};
    dim3 grid(pair_grid(tiles * splits), 1, 1);
    { ScopedKernelEvents ev(LAGA_KERNEL_DW_GEMM, stream); launch_kernel(kernel, grid, dim3(192), L::kTotalBytes, stream, overlap, ta, tb, ta, a); }   // (fp32 atomic epilogue: the output map is unused)
    return launch_status();
}

// ---- packed variable-length sequences ---------------------------------------------------------------
// Host-side plan of one call over packed sequences: every sequence's 128-row tiles in the two orders the
// kernels want (longest work first) and the sequences' starts in the packed tensors and in the padded
// statistics arrays.  `image` is what gets copied to the device, in one piece:
//     int4 q_tiles[n_tiles] | int4 k_tiles[n_tiles] | int2 seqs[n_seqs + 1]
struct SeqPlan {
    int n_seqs = 0, S_total = 0, n_tiles = 0;
    std::vector<int4> image;
    size_t q_tiles_offset() const { return 0; }
    size_t k_tiles_offset() const { return static_cast<size_t>(n_tiles) * sizeof(int4); }
    size_t seqs_offset() const { return 2 * static_cast<size_t>(n_tiles) * sizeof(int4); }
};
// Upper bounds that depend only on (S_total, n_seqs), so that the workspace can be sized without the lengths.
int varlen_s_pad(int S_total, int n_seqs) { return (S_total + 127 * n_seqs + 127) / 128 * 128; }
int varlen_max_tiles(int S_total, int n_seqs) { return S_total / 128 + n_seqs; }
size_t varlen_table_bytes(int S_total, int n_seqs) {
    return align_up(2 * static_cast<size_t>(varlen_max_tiles(S_total, n_seqs)) * sizeof(int4) +
                        (static_cast<size_t>(n_seqs) + 2) / 2 * sizeof(int4),
                    1024);
}

// cu_seqlens: n_seqs + 1 non-decreasing host integers, cu[0] = 0, cu[n_seqs] = S_total.  Empty sequences are
// allowed and contribute nothing.
bool build_seq_plan(const int* cu, int n_seqs, int S_total, bool causal, SeqPlan* plan) {
    if (cu[0] != 0 || cu[n_seqs] != S_total) return false;
    struct Entry { int4 t; int work; };
    std::vector<Entry> q_order, k_order;
    std::vector<int2> seqs(static_cast<size_t>(n_seqs) + 1);
    int pad = 0;
    for (int k = 0; k < n_seqs; ++k) {
        const int len = cu[k + 1] - cu[k];
        if (len < 0) return false;
        seqs[k] = make_int2(cu[k], pad);
        const int tiles = (len + 127) / 128;
        for (int t = 0; t < tiles; ++t) {
            const int4 e = make_int4(cu[k], len, t, pad);
            q_order.push_back({e, causal ? t + 1 : tiles});        // a query tile attends to the key tiles before it
            k_order.push_back({e, causal ? tiles - t : tiles});    // a key tile is attended by the query tiles after it
        }
        pad += tiles * 128;
    }
    seqs[n_seqs] = make_int2(S_total, pad);
    auto by_work = [](const Entry& a, const Entry& b) { return a.work > b.work; };
    std::stable_sort(q_order.begin(), q_order.end(), by_work);
    std::stable_sort(k_order.begin(), k_order.end(), by_work);
    plan->n_seqs = n_seqs;
    plan->S_total = S_total;
    plan->n_tiles = static_cast<int>(q_order.size());
    plan->image.assign(2 * q_order.size() + (seqs.size() + 1) / 2, make_int4(0, 0, 0, 0));
    for (size_t i = 0; i < q_order.size(); ++i) {
        plan->image[i] = q_order[i].t;
        plan->image[q_order.size() + i] = k_order[i].t;
    }
    std::memcpy(plan->image.data() + 2 * q_order.size(), seqs.data(), seqs.size() * sizeof(int2));
    return plan->n_tiles > 0;
}

// Copies the plan into the workspace.  The source is pageable host memory: the runtime stages it before the
// call returns (so the plan may be freed afterwards), at the price of a stream synchronisation inside the call.
int upload_seq_plan(const SeqPlan& plan, void* tables, cudaStream_t stream) {
    return cudaMemcpyAsync(tables, plan.image.data(), plan.image.size() * sizeof(int4), cudaMemcpyHostToDevice, stream) ==
                   cudaSuccess
               ? LAGA_OK
               : LAGA_ERR_CUDA;
}

// ---- Algorithm 1 step 5 -------------------------------------------------------------------------
int launch_attn_fwd(const void* q, const void* kv, const void* k_pe, int S, int h, float softmax_scale,
                    int causal, void* out, float* lse, unsigned* status, cudaStream_t stream,
                    const int4* q_tiles = nullptr, int n_seq_tiles = 0, bool overlap = false) {
    using L = AttnFwdSmem;
    const int N = h * (kDn + kDv);
    CUtensorMap tq, tkv, tpe;   // boxes of 64 columns x one query tile / one key tile of rows
    const uint64_t q_row = static_cast<uint64_t>(h) * (kDn + kDr);
    if (!cached_tmap_bf16(&tq, q, q_row, S, q_row * 2, 128)) return LAGA_ERR_CUDA;
    if (!cached_tmap_bf16(&tkv, kv, N, S, static_cast<uint64_t>(N) * 2, kFwdKeys)) return LAGA_ERR_CUDA;
    if (!cached_tmap_bf16(&tpe, k_pe, kDr, S, kDr * 2, kFwdKeys)) return LAGA_ERR_CUDA;
    const int n_tiles = q_tiles ? n_seq_tiles : (S + 127) / 128;
    AttnFwdArgs a{S, h, softmax_scale * 1.4426950408889634f, reinterpret_cast<const __nv_bfloat16*>(q),
                  reinterpret_cast<__nv_bfloat16*>(out), lse, status,
                  make_schedule(n_tiles, S, h, slot_counter(status, kSlotFwd), q_tiles), slot_probe(status, kSlotFwd)};
    dim3 grid(persistent_grid(n_tiles * h), 1, 1);
    ScopedKernelEvents ev(LAGA_KERNEL_ATTN_FWD, stream);
    launch_kernel(causal ? attn_fwd_sm100_kernel<true> : attn_fwd_sm100_kernel<false>, grid, dim3(kFwdThreads), L::kTotalBytes,
                  stream, overlap, tq, tkv, tpe, a);
    return launch_status();
}

// ---- Section 5.2: backward of step 5 ------------------------------------------------------------
struct BwdWorkspace {
    size_t kv, dkv, stat_l2, stat_delta, dkpe_acc, dk_rope_per_head, dq_acc, tables, total;
    int S_pad;
    int head_window;      // heads per launch of the fused backward; 0 = the two-kernel backward
};

// The fused backward adds dQ tiles into an fp32 accumulator [S][window][192]; the window is the largest
// even split of the heads whose accumulator stays within this budget (so that it, and the Q / dO tiles of
// those heads, stay L2 resident while every key tile sweeps them).
#ifndef LAGA_DQ_ACC_BUDGET_MB
#define LAGA_DQ_ACC_BUDGET_MB 64
#endif
constexpr long long kDqAccBudgetBytes = static_cast<long long>(LAGA_DQ_ACC_BUDGET_MB) << 20;
int fused_head_window(int S, int h) {
    const long long per_head = static_cast<long long>(S) * (kDn + kDr) * sizeof(float);
    long long fit = kDqAccBudgetBytes / per_head;
    if (fit < 1) fit = 1;
    if (fit > h) fit = h;
    const int launches = static_cast<int>((h + fit - 1) / fit);
    return (h + launches - 1) / launches;
}

// n_seqs = 0: one sequence of S tokens; otherwise S tokens in n_seqs packed sequences (tables at the end).
BwdWorkspace bwd_workspace_layout(int S, int h, bool deterministic, bool fused, int n_seqs = 0) {
    BwdWorkspace w;
    const size_t kv_bytes = align_up(static_cast<size_t>(S) * h * (kDn + kDv) * 2, 1024);
    w.S_pad = n_seqs > 0 ? varlen_s_pad(S, n_seqs) : (S + 127) / 128 * 128;
    const size_t stat_bytes = align_up(static_cast<size_t>(h) * w.S_pad * sizeof(float), 1024);
    w.kv = kStatusBytes;
    w.dkv = w.kv + kv_bytes;
    w.stat_l2 = w.dkv + kv_bytes;
    w.stat_delta = w.stat_l2 + stat_bytes;
    w.dkpe_acc = w.stat_delta + stat_bytes;
    w.dk_rope_per_head = w.dkpe_acc + align_up(static_cast<size_t>(S) * kDr * sizeof(float), 1024);
    w.dq_acc = w.dk_rope_per_head +
               (deterministic ? align_up(static_cast<size_t>(h) * S * kDr * sizeof(float), 1024) : 0);
    w.head_window = fused ? fused_head_window(S, h) : 0;
    w.tables = w.dq_acc + align_up(static_cast<size_t>(S) * w.head_window * (kDn + kDr) * sizeof(float), 1024);
    w.total = w.tables + (n_seqs > 0 ? varlen_table_bytes(S, n_seqs) : 0);
    return w;
}

int launch_attn_bwd(const void* q, const void* kv, const void* k_pe, const void* out, const float* lse,
                    const void* dout, int S, int h, float softmax_scale, int causal, void* dq, void* dkv,
                    void* dk_pe, float* stat_l2, float* stat_delta, float* dkpe_acc, float* dk_rope_per_head, int S_pad,
                    float* dq_acc, int head_window, unsigned* status, cudaStream_t stream,
                    const int4* q_tiles = nullptr, const int4* k_tiles = nullptr, const int2* seqs = nullptr,
                    int n_seqs = 0, int n_seq_tiles = 0, bool overlap = false,
                    const void* rebuild_c_kv = nullptr, const void* rebuild_w = nullptr) {
    const int N = h * (kDn + kDv);
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    {   // delta and the transposed, padded softmax statistics; clears the rope-gradient accumulator on the way
        const long long items = static_cast<long long>(S_pad) * h;   // eight lanes per (row, head)
        const unsigned blocks = static_cast<unsigned>((items * 8 + 255) / 256);
        ScopedKernelEvents ev(LAGA_KERNEL_BWD_DELTA, stream);
        launch_kernel(bwd_delta_kernel, dim3(blocks), dim3(256), 0, stream, overlap, reinterpret_cast<const __nv_bfloat16*>(out),
                      reinterpret_cast<const __nv_bfloat16*>(dout), lse, S, h, S_pad, stat_l2, stat_delta,
                      reinterpret_cast<float4*>(dkpe_acc), static_cast<size_t>(S) * kDr / 4, seqs, n_seqs);
        if (launch_status() != LAGA_OK) return LAGA_ERR_CUDA;
    }
    const uint64_t q_row = static_cast<uint64_t>(h) * 192, do_row = static_cast<uint64_t>(h) * 128;
    CUtensorMap tq, tkv, tpe, tdo;   // boxes of 64 columns x 128 rows
    if (!cached_tmap_bf16(&tq, q, q_row, S, q_row * 2, 128) || !cached_tmap_bf16(&tdo, dout, do_row, S, do_row * 2, 128) ||
        !cached_tmap_bf16(&tkv, kv, N, S, static_cast<uint64_t>(N) * 2, 128) ||
        !cached_tmap_bf16(&tpe, k_pe, kDr, S, kDr * 2, 128))
        return LAGA_ERR_CUDA;
    const int n_tiles = q_tiles ? n_seq_tiles : (S + 127) / 128;
    if (head_window > 0) {
        // One pass over the score tiles on CTA pairs, a window of heads per launch; dQ goes through dq_acc.
        if (cudaMemsetAsync(dq_acc, 0, static_cast<size_t>(S) * head_window * (kDn + kDr) * sizeof(float), stream) != cudaSuccess)
            return LAGA_ERR_CUDA;
        const int pairs_max = fused_pair_count();
        for (int head_begin = 0; head_begin < h; head_begin += head_window) {
            const int head_count = h - head_begin < head_window ? h - head_begin : head_window;
            const int items = n_tiles * head_count;
            dim3 grid(2u * static_cast<unsigned>(items < pairs_max ? items : pairs_max), 1, 1);
            AttnBwdFusedArgs f{S, h, S_pad, head_begin, head_count, scale_log2, softmax_scale, stat_l2, stat_delta,
                               reinterpret_cast<const __nv_bfloat16*>(kv), reinterpret_cast<__nv_bfloat16*>(dkv), dkpe_acc,
                               dq_acc, status, slot_probe(status, kSlotFused)};
            {
                ScopedKernelEvents ev(LAGA_KERNEL_ATTN_BWD_FUSED, stream);
                if (causal) attn_bwd_fused_sm100_kernel<true><<<grid, kBwdThreads, AttnBwdFusedSmem::kTotalBytes, stream>>>(tq, tdo, tkv, tpe, f);
                else attn_bwd_fused_sm100_kernel<false><<<grid, kBwdThreads, AttnBwdFusedSmem::kTotalBytes, stream>>>(tq, tdo, tkv, tpe, f);
            }
            if (launch_status() != LAGA_OK) return LAGA_ERR_CUDA;
            {
                const size_t n = static_cast<size_t>(S) * head_count * (kDn + kDr) / 8;
                ScopedKernelEvents ev(LAGA_KERNEL_DQ_CONVERT, stream);
                bwd_dq_convert_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(
                    dq_acc, S, h, head_begin, head_count, softmax_scale, reinterpret_cast<__nv_bfloat16*>(dq));
            }
            if (launch_status() != LAGA_OK) return LAGA_ERR_CUDA;
        }
    } else {
        dim3 grid(persistent_grid(n_tiles * h), 1, 1);
        AttnBwdDkvArgs a{S, h, S_pad, scale_log2, softmax_scale, stat_l2, stat_delta,
                         reinterpret_cast<__nv_bfloat16*>(dkv), dkpe_acc, dk_rope_per_head, status,
                         make_schedule(n_tiles, S, h, slot_counter(status, kSlotDkv), k_tiles), slot_probe(status, kSlotDkv)};
        AttnBwdDqArgs b{S, h, scale_log2, softmax_scale, lse, stat_delta, S_pad,
                        reinterpret_cast<const __nv_bfloat16*>(dout), reinterpret_cast<__nv_bfloat16*>(dq), status,
                        make_schedule(n_tiles, S, h, slot_counter(status, kSlotDq), q_tiles), slot_probe(status, kSlotDq)};
        {
            ScopedKernelEvents ev(LAGA_KERNEL_ATTN_BWD_DKV, stream);
            if (rebuild_c_kv != nullptr) {     // step 4 inside the kernel: boxes of the latent (64 x 128 rows) and of W (64 x 64 rows)
                CUtensorMap tc, tw;
                if (!cached_tmap_bf16(&tc, rebuild_c_kv, kDc, S, kDc * 2, 128) ||
                    !cached_tmap_bf16(&tw, rebuild_w, N, kDc, static_cast<uint64_t>(N) * 2, 64))
                    return LAGA_ERR_CUDA;
                launch_kernel(causal ? attn_bwd_dkv_sm100_kernel<true, true> : attn_bwd_dkv_sm100_kernel<false, true>, grid,
                              dim3(kBwdThreads), AttnBwdDkvSmem::kTotalBytes, stream, true, tq, tdo, tkv, tpe, tc, tw, a);
            } else {
                launch_kernel(causal ? attn_bwd_dkv_sm100_kernel<true, false> : attn_bwd_dkv_sm100_kernel<false, false>, grid,
                              dim3(kBwdThreads), AttnBwdDkvSmem::kTotalBytes, stream, true, tq, tdo, tkv, tpe, tkv, tkv, a);
            }
        }
        if (launch_status() != LAGA_OK) return LAGA_ERR_CUDA;
        {
            ScopedKernelEvents ev(LAGA_KERNEL_ATTN_BWD_DQ, stream);
            launch_kernel(causal ? attn_bwd_dq_sm100_kernel<true> : attn_bwd_dq_sm100_kernel<false>, grid, dim3(kBwdThreads),
                          AttnBwdDqSmem::kTotalBytes, stream, true, tq, tdo, tkv, tpe, b);
        }
    }
    if (launch_status() != LAGA_OK) return LAGA_ERR_CUDA;
    {
        ScopedKernelEvents ev(LAGA_KERNEL_DKPE_REDUCE, stream);
        if (dk_rope_per_head != nullptr) {
            const size_t n = static_cast<size_t>(S) * kDr;
            launch_kernel(bwd_dkpe_reduce_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, stream, true,
                          dk_rope_per_head, S, h, reinterpret_cast<__nv_bfloat16*>(dk_pe));
        } else {
            const size_t n = static_cast<size_t>(S) * kDr / 4;
            launch_kernel(bwd_dkpe_convert_kernel, dim3(static_cast<unsigned>((n + 255) / 256)), dim3(256), 0, stream, true,
                          dkpe_acc, S, reinterpret_cast<__nv_bfloat16*>(dk_pe));
        }
    }
    return launch_status();
}

// ---- absorbed form (Section 3.2, baseline B2): comparison path --------------------------------------
// q_abs[S, h, d_c] = q_nope[S, h, d_n] . W_uk[h]^T, batched over the heads: head i reads columns
// [192 i, 192 i + 128) of q and columns [256 i, 256 i + 128) of W (rows = latent index = the GEMM's N).
int launch_q_absorb(const void* q, const void* w, int S, int h, void* q_abs, unsigned* status, cudaStream_t stream) {
    constexpr int BN = 256, STAGES = kGemmStages;
    auto kernel = gemm_pair_sm100_kernel<BN, STAGES, false, false, EPI_BF16>;
    using L = GemmPairSmem<BN, STAGES>;
    const uint64_t q_row = static_cast<uint64_t>(h) * (kDn + kDr), w_row = static_cast<uint64_t>(h) * (kDn + kDv);
    CUtensorMap ta, tb;
    if (!cached_tmap_bf16(&ta, q, q_row, S, q_row * 2, 128)) return LAGA_ERR_CUDA;
    if (!cached_tmap_bf16(&tb, w, w_row, kDc, w_row * 2, BN / 2)) return LAGA_ERR_CUDA;
    CUtensorMap tc;
    const uint64_t qa_row = static_cast<uint64_t>(h) * kDc;
    if (!cached_tmap_bf16(&tc, q_abs, qa_row, S, qa_row * 2, 32)) return LAGA_ERR_CUDA;
    GemmArgs a{S, kDc, kDn, kDn / 64, 1, q_abs, h * kDc, status, nullptr, 0, h, kDn + kDr, kDn + kDv, kDc};
    dim3 grid(pair_grid((kDc / BN) * ((S + 255) / 256) * h), 1, 1);
    { ScopedKernelEvents ev(LAGA_KERNEL_Q_ABSORB, stream); kernel<<<grid, 192, L::kTotalBytes, stream>>>(ta, tb, tc, a); }
    return launch_status();
}

// out[S, h, d_v] = o_lat[S, h, d_c] . W_uv[h], batched over the heads: head i reads columns
// [512 i, 512 i + 512) of o_lat and columns [256 i + 128, 256 i + 256) of W (rows = latent index = the GEMM's K).
int launch_v_project(const void* o_lat, const void* w, int S, int h, void* out, unsigned* status, cudaStream_t stream) {
    constexpr int BN = 128, STAGES = 4;
    auto kernel = gemm_sm100_kernel<BN, STAGES, false, true, EPI_BF16>;
    using L = GemmSmem<BN, STAGES>;
    const uint64_t o_row = static_cast<uint64_t>(h) * kDc, w_row = static_cast<uint64_t>(h) * (kDn + kDv);
    CUtensorMap ta, tb;
    if (!cached_tmap_bf16(&ta, o_lat, o_row, S, o_row * 2, 128)) return LAGA_ERR_CUDA;
    // the map starts at W's column d_nope: column 0 of the map is V channel 0 of head 0
    if (!cached_tmap_bf16(&tb, static_cast<const uint8_t*>(w) + kDn * 2, w_row - kDn, kDc, w_row * 2, 64)) return LAGA_ERR_CUDA;
    GemmArgs a{S, kDv, kDc, kDc / 64, 1, out, h * kDv, status, nullptr, 0, h, kDc, kDn + kDv, kDv};
    dim3 grid(persistent_grid(((S + 127) / 128) * h), 1, 1);
    { ScopedKernelEvents ev(LAGA_KERNEL_V_PROJECT, stream); kernel<<<grid, 192, L::kTotalBytes, stream>>>(ta, tb, a); }
    return launch_status();
}

int launch_attn_absorbed(const void* q, const void* q_abs, const void* c_kv, const void* k_pe, int S, int h,
                         float softmax_scale, int causal, void* o_lat, float* lse, unsigned* status, cudaStream_t stream) {
    using L = AttnAbsorbedSmem;
    const uint64_t qa_row = static_cast<uint64_t>(h) * kDc, q_row = static_cast<uint64_t>(h) * (kDn + kDr);
    CUtensorMap tqa, tq, tc, tpe;
    if (!cached_tmap_bf16(&tqa, q_abs, qa_row, S, qa_row * 2, 128) || !cached_tmap_bf16(&tq, q, q_row, S, q_row * 2, 128) ||
        !cached_tmap_bf16(&tc, c_kv, kDc, S, kDc * 2, kAbsKeys) || !cached_tmap_bf16(&tpe, k_pe, kDr, S, kDr * 2, kAbsKeys))
        return LAGA_ERR_CUDA;
    AttnAbsorbedArgs a{S, h, softmax_scale * 1.4426950408889634f, reinterpret_cast<const __nv_bfloat16*>(q_abs),
                       reinterpret_cast<__nv_bfloat16*>(o_lat), lse, status};
    dim3 grid((S + 127) / 128, 2 * h, 1);
    ScopedKernelEvents ev(LAGA_KERNEL_ATTN_ABSORBED, stream);
    if (causal) attn_absorbed_fwd_sm100_kernel<true><<<grid, kAbsThreads, L::kTotalBytes, stream>>>(tqa, tq, tc, tpe, a);
    else attn_absorbed_fwd_sm100_kernel<false><<<grid, kAbsThreads, L::kTotalBytes, stream>>>(tqa, tq, tc, tpe, a);
    return launch_status();
}

// Self-test of the bounded-wait machinery every kernel here relies on: two warps wait on an mbarrier
// that nothing will ever arrive on.  After `budget_ns` the first waiter records the site in the status
// word and raises the abort flag, the other waiter sees the flag, and the CTA exits normally.
__global__ void selftest_bounded_wait_kernel(unsigned* status, unsigned long long budget_ns) {
    __shared__ uint64_t never_signalled;
    __shared__ AbortFlag abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&never_signalled, 1);
        abort_flag.value = 0;
        mbar_fence_init();
    }
    __syncthreads();
    const bool ok = mbar_wait_warp(&never_signalled, 0, &abort_flag, status, 0x7e57u, budget_ns);
    if (ok && threadIdx.x == 0) atomicExch(status, 0xdeadu);   // cannot happen: nothing arrives
}

// Clears the status word and the work counters of a workspace's status slot.
int zero_status(void* status_slot, cudaStream_t stream) {
    return cudaMemsetAsync(status_slot, 0, kStatusClearBytes, stream) == cudaSuccess ? LAGA_OK : LAGA_ERR_CUDA;
}
// A bare status word handed to a step entry point (no counters behind it).
int zero_status_word(void* status_word, cudaStream_t stream) {
    return cudaMemsetAsync(status_word, 0, sizeof(unsigned), stream) == cudaSuccess ? LAGA_OK : LAGA_ERR_CUDA;
}

}  // namespace

extern "C" {

int laga_version(void) { return 211; }

const char* laga_status_string(int status) {
    switch (status) {
        case LAGA_OK: return "LAGA_OK";
        case LAGA_ERR_INVALID_ARG: return "LAGA_ERR_INVALID_ARG";
        case LAGA_ERR_UNSUPPORTED: return "LAGA_ERR_UNSUPPORTED";
        case LAGA_ERR_WORKSPACE_TOO_SMALL: return "LAGA_ERR_WORKSPACE_TOO_SMALL";
        case LAGA_ERR_CUDA: return "LAGA_ERR_CUDA";
        case LAGA_ERR_DEVICE_TIMEOUT: return "LAGA_ERR_DEVICE_TIMEOUT";
        case LAGA_ERR_DEVICE_CHECK: return "LAGA_ERR_DEVICE_CHECK";
        default: return "LAGA_ERR_UNKNOWN";
    }
}

size_t laga_fwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v) {
    if (S < 1 || h < 1 || !geometry_supported(d_c, d_nope, d_rope, d_v)) return 0;
    return kStatusBytes + align_up(static_cast<size_t>(S) * h * (d_nope + d_v) * 2, 1024);
}

size_t laga_bwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v, unsigned flags) {
    if (S < 1 || h < 1 || !geometry_supported(d_c, d_nope, d_rope, d_v)) return 0;
    return bwd_workspace_layout(S, h, (flags & LAGA_FLAG_DETERMINISTIC) != 0, (flags & LAGA_FLAG_FUSED_BWD) != 0).total;
}

int laga_up_project(const void* c_kv, const void* w_kv_b, int S, int h, int d_c, int d_nope, int d_v, void* kv,
                    void* status_word, void* stream) {
    if (!c_kv || !w_kv_b || !kv || !status_word || S < 1 || h < 1) return LAGA_ERR_INVALID_ARG;
    if (!aligned16(c_kv) || !aligned16(w_kv_b) || !aligned16(kv)) return LAGA_ERR_INVALID_ARG;
    if (!geometry_supported(d_c, d_nope, kDr, d_v)) return LAGA_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({c_kv, w_kv_b, kv, status_word})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = zero_status_word(status_word, st)) != LAGA_OK) return rc;
    return launch_up_project(c_kv, w_kv_b, S, h * (kDn + kDv), kv, static_cast<unsigned*>(status_word), st, false, d_c);
}

int laga_kv_backward(const void* dkv, const void* c_kv, const void* w_kv_b, int S, int h, int d_c, int d_nope,
                     int d_v, void* dc_kv, float* dw_kv_b, unsigned flags, void* status_word, void* stream) {
    if (!dkv || !c_kv || !w_kv_b || !dc_kv || !dw_kv_b || !status_word || S < 1 || h < 1)
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(dkv) || !aligned16(c_kv) || !aligned16(w_kv_b) || !aligned16(dc_kv) || !aligned16(dw_kv_b))
        return LAGA_ERR_INVALID_ARG;
    if (flags & ~(LAGA_FLAG_ACCUM_DW | LAGA_FLAG_DETERMINISTIC)) return LAGA_ERR_INVALID_ARG;
    if (!geometry_supported(d_c, d_nope, kDr, d_v)) return LAGA_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({dkv, c_kv, w_kv_b, dc_kv, dw_kv_b, status_word})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* status = static_cast<unsigned*>(status_word);
    const int N = h * (kDn + kDv);
    const bool accumulate = (flags & LAGA_FLAG_ACCUM_DW) != 0;
    if ((rc = zero_status_word(status_word, st)) != LAGA_OK) return rc;
    if ((rc = launch_dckv(dkv, w_kv_b, S, N, dc_kv, accumulate ? nullptr : dw_kv_b,
                          accumulate ? 0 : static_cast<size_t>(d_c) * N, status, st, false, d_c)) != LAGA_OK)
        return rc;
    return launch_dw(c_kv, dkv, S, N, dw_kv_b, (flags & LAGA_FLAG_DETERMINISTIC) != 0, status, st, false, d_c);
}

// laga_fwd and laga_fwd_varlen: cu_seqlens == nullptr means one sequence of S tokens.
static int fwd_impl(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const int* cu_seqlens, int n_seqs,
                    int S, int h, int d_c, int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out,
                    float* lse, void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !out || !lse || !workspace || S < 1 || h < 1)
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(c_kv) || !aligned16(k_pe) || !aligned16(w_kv_b) || !aligned16(out) ||
        !aligned16(lse) || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return LAGA_ERR_INVALID_ARG;
    if (flags != 0 || !(softmax_scale > 0.f)) return LAGA_ERR_INVALID_ARG;
    if (!geometry_supported(d_c, d_nope, d_rope, d_v)) return LAGA_ERR_UNSUPPORTED;
    const size_t kv_end = laga_fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v);
    SeqPlan plan;
    if (cu_seqlens != nullptr) {
        if (n_seqs < 1 || !build_seq_plan(cu_seqlens, n_seqs, S, causal != 0, &plan)) return LAGA_ERR_INVALID_ARG;
        if (workspace_bytes < kv_end + varlen_table_bytes(S, n_seqs)) return LAGA_ERR_WORKSPACE_TOO_SMALL;
    } else if (workspace_bytes < kv_end) {
        return LAGA_ERR_WORKSPACE_TOO_SMALL;
    }
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({q, c_kv, k_pe, w_kv_b, out, lse, workspace})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* status = static_cast<unsigned*>(workspace);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    void* kv = base + kStatusBytes;
    if ((rc = zero_status(status, st)) != LAGA_OK) return rc;
    const int4* q_tiles = nullptr;
    if (cu_seqlens != nullptr) {
        if ((rc = upload_seq_plan(plan, base + kv_end, st)) != LAGA_OK) return rc;
        q_tiles = reinterpret_cast<const int4*>(base + kv_end + plan.q_tiles_offset());
    }
    // step 4 is token-wise: one GEMM over all the packed tokens
    if ((rc = launch_up_project(c_kv, w_kv_b, S, h * (kDn + kDv), kv, status, st, false, d_c)) != LAGA_OK) return rc;
    return launch_attn_fwd(q, kv, k_pe, S, h, softmax_scale, causal, out, lse, status, st, q_tiles, plan.n_tiles, true);
}

int laga_fwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S, int h, int d_c,
             int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out, float* lse,
             void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    return fwd_impl(q, c_kv, k_pe, w_kv_b, nullptr, 0, S, h, d_c, d_nope, d_rope, d_v, softmax_scale, causal, out, lse,
                    workspace, workspace_bytes, flags, stream);
}

size_t laga_fwd_varlen_workspace_bytes(int S_total, int n_seqs, int h, int d_c, int d_nope, int d_rope, int d_v) {
    const size_t base = laga_fwd_workspace_bytes(S_total, h, d_c, d_nope, d_rope, d_v);
    if (base == 0 || n_seqs < 1) return 0;
    return base + varlen_table_bytes(S_total, n_seqs);
}

size_t laga_bwd_varlen_workspace_bytes(int S_total, int n_seqs, int h, int d_c, int d_nope, int d_rope, int d_v,
                                       unsigned flags) {
    if (S_total < 1 || h < 1 || n_seqs < 1 || !geometry_supported(d_c, d_nope, d_rope, d_v)) return 0;
    if (flags & LAGA_FLAG_FUSED_BWD) return 0;
    return bwd_workspace_layout(S_total, h, (flags & LAGA_FLAG_DETERMINISTIC) != 0, false, n_seqs).total;
}

int laga_linear(const void* x, const void* w, int M, int K, int N, void* y, void* status_word, void* stream) {
    if (!x || !w || !y || !status_word || M < 1 || K < 8 || N < 8 || (K & 7) || (N & 7)) return LAGA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return LAGA_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({x, w, y, status_word})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = zero_status_word(status_word, st)) != LAGA_OK) return rc;
    return launch_up_project(x, w, M, N, y, static_cast<unsigned*>(status_word), st, false, K);
}

int laga_linear_backward(const void* dy, const void* x, const void* w, int M, int K, int N, void* dx, float* dw,
                         unsigned flags, void* status_word, void* stream) {
    if (!dy || !x || !w || !dx || !dw || !status_word || M < 1 || K < 8 || N < 8 || (K & 7) || (N & 7))
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(dy) || !aligned16(x) || !aligned16(w) || !aligned16(dx) || !aligned16(dw)) return LAGA_ERR_INVALID_ARG;
    if (flags & ~(LAGA_FLAG_ACCUM_DW | LAGA_FLAG_DETERMINISTIC)) return LAGA_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({dy, x, w, dx, dw, status_word})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* status = static_cast<unsigned*>(status_word);
    const bool accumulate = (flags & LAGA_FLAG_ACCUM_DW) != 0;
    if ((rc = zero_status_word(status_word, st)) != LAGA_OK) return rc;
    if ((rc = launch_dckv(dy, w, M, N, dx, accumulate ? nullptr : dw, accumulate ? 0 : static_cast<size_t>(K) * N, status, st,
                          false, K)) != LAGA_OK)
        return rc;
    return launch_dw(x, dy, M, N, dw, (flags & LAGA_FLAG_DETERMINISTIC) != 0, status, st, true, K);
}

int laga_layernorm(const void* x, const void* gamma, const void* beta, int M, int D, float eps, void* y, float* mean,
                   float* rstd, void* stream) {
    if (!x || !gamma || !y || M < 1 || D < 8 || (D & 7) || D > kLnMaxD || !(eps >= 0.f)) return LAGA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(y) || (beta && !aligned16(beta))) return LAGA_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({x, gamma, y})) != LAGA_OK) return rc;
    if (beta && (rc = check_pointers({beta})) != LAGA_OK) return rc;
    if (mean && (rc = check_pointers({mean})) != LAGA_OK) return rc;
    if (rstd && (rc = check_pointers({rstd})) != LAGA_OK) return rc;
    // one resident wave striding over the rows (four blocks of 256 threads fit an SM at D <= 512)
    const int blocks_needed = (M + kLnWarps - 1) / kLnWarps, cap = sm_count() * 4;
    const dim3 grid(blocks_needed < cap ? blocks_needed : cap), block(kLnWarps * 32);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto xs = static_cast<const __nv_bfloat16*>(x), gs = static_cast<const __nv_bfloat16*>(gamma), bs = static_cast<const __nv_bfloat16*>(beta);
    auto ys = static_cast<__nv_bfloat16*>(y);
    if (D <= 256) layernorm_fwd_kernel<1><<<grid, block, 0, st>>>(xs, gs, bs, M, D, eps, ys, mean, rstd);
    else if (D <= 512) layernorm_fwd_kernel<2><<<grid, block, 0, st>>>(xs, gs, bs, M, D, eps, ys, mean, rstd);
    else layernorm_fwd_kernel<4><<<grid, block, 0, st>>>(xs, gs, bs, M, D, eps, ys, mean, rstd);
    return launch_status();
}

int laga_layernorm_backward(const void* dy, const void* x, const void* gamma, const float* mean, const float* rstd, int M,
                            int D, void* dx, float* dgamma, float* dbeta, void* stream) {
    if (!dy || !x || !gamma || !mean || !rstd || !dx || !dgamma || M < 1 || D < 8 || (D & 7) || D > kLnMaxD)
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(dy) || !aligned16(x) || !aligned16(gamma) || !aligned16(dx)) return LAGA_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({dy, x, gamma, mean, rstd, dx, dgamma})) != LAGA_OK) return rc;
    if (dbeta && (rc = check_pointers({dbeta})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(dgamma, 0, static_cast<size_t>(D) * sizeof(float), st) != cudaSuccess) return LAGA_ERR_CUDA;
    if (dbeta && cudaMemsetAsync(dbeta, 0, static_cast<size_t>(D) * sizeof(float), st) != cudaSuccess) return LAGA_ERR_CUDA;
    // one resident wave (two blocks per SM) strides over the rows: each block ends with D atomics per output
    const int blocks_needed = (M + kLnWarps - 1) / kLnWarps, cap = sm_count() * 2;
    const dim3 grid(blocks_needed < cap ? blocks_needed : cap), block(kLnWarps * 32);
    auto dys = static_cast<const __nv_bfloat16*>(dy), xs = static_cast<const __nv_bfloat16*>(x), gs = static_cast<const __nv_bfloat16*>(gamma);
    auto dxs = static_cast<__nv_bfloat16*>(dx);
    if (D <= 256) layernorm_bwd_kernel<1><<<grid, block, 0, st>>>(dys, xs, gs, mean, rstd, M, D, dxs, dgamma, dbeta);
    else if (D <= 512) layernorm_bwd_kernel<2><<<grid, block, 0, st>>>(dys, xs, gs, mean, rstd, M, D, dxs, dgamma, dbeta);
    else layernorm_bwd_kernel<4><<<grid, block, 0, st>>>(dys, xs, gs, mean, rstd, M, D, dxs, dgamma, dbeta);
    return launch_status();
}

int laga_fwd_varlen(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const int* cu_seqlens,
                    int n_seqs, int S_total, int h, int d_c, int d_nope, int d_rope, int d_v, float softmax_scale,
                    int causal, void* out, float* lse, void* workspace, size_t workspace_bytes, unsigned flags,
                    void* stream) {
    if (!cu_seqlens) return LAGA_ERR_INVALID_ARG;
    return fwd_impl(q, c_kv, k_pe, w_kv_b, cu_seqlens, n_seqs, S_total, h, d_c, d_nope, d_rope, d_v, softmax_scale, causal,
                    out, lse, workspace, workspace_bytes, flags, stream);
}

// laga_bwd and laga_bwd_varlen: cu_seqlens == nullptr means one sequence of S tokens.
static int bwd_impl(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const void* out, const float* lse,
                    const void* dout, const int* cu_seqlens, int n_seqs, int S, int h, int d_c, int d_nope, int d_rope,
                    int d_v, float softmax_scale, int causal, void* dq, void* dc_kv, void* dk_pe, float* dw_kv_b,
                    void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !out || !lse || !dout || !dq || !dc_kv || !dk_pe || !dw_kv_b ||
        !workspace || S < 1 || h < 1)
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(c_kv) || !aligned16(k_pe) || !aligned16(w_kv_b) || !aligned16(out) ||
        !aligned16(lse) || !aligned16(dout) || !aligned16(dq) || !aligned16(dc_kv) || !aligned16(dk_pe) ||
        !aligned16(dw_kv_b) || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return LAGA_ERR_INVALID_ARG;
    if ((flags & ~(LAGA_FLAG_ACCUM_DW | LAGA_FLAG_DETERMINISTIC | LAGA_FLAG_KV_SAVED | LAGA_FLAG_FUSED_BWD | LAGA_FLAG_FUSED_KV_REBUILD)) ||
        !(softmax_scale > 0.f))
        return LAGA_ERR_INVALID_ARG;
    if (!geometry_supported(d_c, d_nope, d_rope, d_v)) return LAGA_ERR_UNSUPPORTED;
    const bool rebuild = (flags & LAGA_FLAG_FUSED_KV_REBUILD) != 0;
    if (rebuild && (flags & (LAGA_FLAG_KV_SAVED | LAGA_FLAG_FUSED_BWD))) return LAGA_ERR_INVALID_ARG;
    if (rebuild && !geometry_is_v3(d_c, d_nope, d_rope, d_v)) return LAGA_ERR_UNSUPPORTED;   // eight 64-deep chunks
    const bool deterministic = (flags & LAGA_FLAG_DETERMINISTIC) != 0;
    const bool accumulate = (flags & LAGA_FLAG_ACCUM_DW) != 0;
    const bool fused = (flags & LAGA_FLAG_FUSED_BWD) != 0;
    if (fused && deterministic) return LAGA_ERR_INVALID_ARG;   // the fused kernel's dQ and dk_pe sums are order dependent
    if (fused && cu_seqlens != nullptr) return LAGA_ERR_INVALID_ARG;   // the one-pass kernel takes one sequence
    SeqPlan plan;
    if (cu_seqlens != nullptr && (n_seqs < 1 || !build_seq_plan(cu_seqlens, n_seqs, S, causal != 0, &plan)))
        return LAGA_ERR_INVALID_ARG;
    const BwdWorkspace w = bwd_workspace_layout(S, h, deterministic, fused, cu_seqlens ? n_seqs : 0);
    if (workspace_bytes < w.total) return LAGA_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({q, c_kv, k_pe, w_kv_b, out, lse, dout, dq, dc_kv, dk_pe, dw_kv_b, workspace})) != LAGA_OK)
        return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    unsigned* status = reinterpret_cast<unsigned*>(base);
    void* kv = base + w.kv;
    void* dkv = base + w.dkv;
    const int N = h * (kDn + kDv);
    if ((rc = zero_status(status, st)) != LAGA_OK) return rc;
    const int4 *q_tiles = nullptr, *k_tiles = nullptr;
    const int2* seqs = nullptr;
    if (cu_seqlens != nullptr) {
        if ((rc = upload_seq_plan(plan, base + w.tables, st)) != LAGA_OK) return rc;
        q_tiles = reinterpret_cast<const int4*>(base + w.tables + plan.q_tiles_offset());
        k_tiles = reinterpret_cast<const int4*>(base + w.tables + plan.k_tiles_offset());
        seqs = reinterpret_cast<const int2*>(base + w.tables + plan.seqs_offset());
    }
    // K_nope / V are recomputed from the latent (the forward keeps only out and lse) unless the caller
    // vouches that the forward's copy is still in this workspace: both layouts put it right after the status.
    // (or the dK/dV kernel rebuilds them tile by tile: LAGA_FLAG_FUSED_KV_REBUILD)
    const bool up_project = !(flags & LAGA_FLAG_KV_SAVED) && !rebuild;
    if (up_project && (rc = launch_up_project(c_kv, w_kv_b, S, N, kv, status, st, false, d_c)) != LAGA_OK) return rc;
    if ((rc = launch_attn_bwd(q, kv, k_pe, out, lse, dout, S, h, softmax_scale, causal, dq, dkv, dk_pe,
                              reinterpret_cast<float*>(base + w.stat_l2), reinterpret_cast<float*>(base + w.stat_delta),
                              reinterpret_cast<float*>(base + w.dkpe_acc),
                              deterministic ? reinterpret_cast<float*>(base + w.dk_rope_per_head) : nullptr, w.S_pad,
                              reinterpret_cast<float*>(base + w.dq_acc), w.head_window, status, st, q_tiles, k_tiles, seqs,
                              plan.n_seqs, plan.n_tiles, /*overlap=*/up_project, rebuild ? c_kv : nullptr, w_kv_b)) != LAGA_OK)
        return rc;
    // the two GEMMs of Section 5.2 are token-wise: one launch each over all the packed tokens
    if ((rc = launch_dckv(dkv, w_kv_b, S, N, dc_kv, accumulate ? nullptr : dw_kv_b,
                          accumulate ? 0 : static_cast<size_t>(d_c) * N, status, st, true, d_c)) != LAGA_OK)
        return rc;
    return launch_dw(c_kv, dkv, S, N, dw_kv_b, deterministic, status, st, true, d_c);
}

int laga_bwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const void* out,
             const float* lse, const void* dout, int S, int h, int d_c, int d_nope, int d_rope, int d_v,
             float softmax_scale, int causal, void* dq, void* dc_kv, void* dk_pe, float* dw_kv_b, void* workspace,
             size_t workspace_bytes, unsigned flags, void* stream) {
    return bwd_impl(q, c_kv, k_pe, w_kv_b, out, lse, dout, nullptr, 0, S, h, d_c, d_nope, d_rope, d_v, softmax_scale, causal,
                    dq, dc_kv, dk_pe, dw_kv_b, workspace, workspace_bytes, flags, stream);
}

int laga_bwd_varlen(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const void* out,
                    const float* lse, const void* dout, const int* cu_seqlens, int n_seqs, int S_total, int h, int d_c,
                    int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* dq, void* dc_kv, void* dk_pe,
                    float* dw_kv_b, void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!cu_seqlens) return LAGA_ERR_INVALID_ARG;
    return bwd_impl(q, c_kv, k_pe, w_kv_b, out, lse, dout, cu_seqlens, n_seqs, S_total, h, d_c, d_nope, d_rope, d_v,
                    softmax_scale, causal, dq, dc_kv, dk_pe, dw_kv_b, workspace, workspace_bytes, flags, stream);
}

// ---- forward without caller-provided scratch ----------------------------------------------------
// Scratch for laga_fwd_builtin_scratch: the launch status slot followed by the bf16 up-projection
// KV[S, h*256].  It lives in the library image, so every GPU that loads the library holds these
// bytes until the process exits; the cap keeps that cost modest.
constexpr size_t kBuiltinKvBytes = size_t(16) << 20;                       // S * h <= 32768
static __device__ __align__(256) unsigned char g_builtin_scratch[kStatusBytes + kBuiltinKvBytes];

// Device address of g_builtin_scratch on the current device.  In host code the symbol's name is only
// a handle, never an address a kernel may use: the address comes from cudaGetSymbolAddress, looked up
// once per device with that device current.
static void lookup_builtin_scratch(DeviceInfo* info) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_builtin_scratch) != cudaSuccess || !p) {
        (void)cudaGetLastError();
        return;
    }
    info->builtin_scratch = static_cast<unsigned char*>(p);
}

static int builtin_scratch_address(unsigned char** ptr) {
    DeviceInfo* info = nullptr;
    const int rc = current_device(&info);
    if (rc != LAGA_OK) return rc;
    std::call_once(info->scratch_once, lookup_builtin_scratch, info);
    if (!info->builtin_scratch) return LAGA_ERR_CUDA;
    *ptr = info->builtin_scratch;
    return LAGA_OK;
}

int laga_fwd_builtin_scratch(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S, int h,
                             int d_c, int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out,
                             float* lse, void* stream) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !out || !lse || S < 1 || h < 1) return LAGA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(c_kv) || !aligned16(k_pe) || !aligned16(w_kv_b) || !aligned16(out) ||
        !aligned16(lse))
        return LAGA_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f)) return LAGA_ERR_INVALID_ARG;
    if (!geometry_supported(d_c, d_nope, d_rope, d_v)) return LAGA_ERR_UNSUPPORTED;
    // the built-in scratch is a fixed size: larger problems must bring their own workspace (laga_fwd)
    if (static_cast<size_t>(S) * h * (kDn + kDv) * 2 > kBuiltinKvBytes) return LAGA_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({q, c_kv, k_pe, w_kv_b, out, lse})) != LAGA_OK) return rc;
    unsigned char* base = nullptr;
    if ((rc = builtin_scratch_address(&base)) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* status = reinterpret_cast<unsigned*>(base);
    void* kv = base + kStatusBytes;
    // The array keeps whatever the previous call left: the status slot (status word and work counter) must
    // start at zero; KV rows [0, S) are fully overwritten by the up-projection before the attention kernel
    // reads them.
    if ((rc = zero_status(status, st)) != LAGA_OK) return rc;
    if ((rc = launch_up_project(c_kv, w_kv_b, S, h * (kDn + kDv), kv, status, st, false, d_c)) != LAGA_OK) return rc;
    return launch_attn_fwd(q, kv, k_pe, S, h, softmax_scale, causal, out, lse, status, st, nullptr, 0, true);
}

size_t laga_absorbed_fwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v) {
    if (S < 1 || h < 1 || !geometry_is_v3(d_c, d_nope, d_rope, d_v)) return 0;
    return kStatusBytes + 2 * align_up(static_cast<size_t>(S) * h * d_c * 2, 1024);
}

int laga_absorbed_fwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S, int h, int d_c,
                      int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out, float* lse,
                      void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !out || !lse || !workspace || S < 1 || h < 1)
        return LAGA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(c_kv) || !aligned16(k_pe) || !aligned16(w_kv_b) || !aligned16(out) ||
        !aligned16(lse) || (reinterpret_cast<uintptr_t>(workspace) & 1023u))
        return LAGA_ERR_INVALID_ARG;
    if (flags != 0 || !(softmax_scale > 0.f)) return LAGA_ERR_INVALID_ARG;
    if (!geometry_is_v3(d_c, d_nope, d_rope, d_v)) return LAGA_ERR_UNSUPPORTED;
    if (workspace_bytes < laga_absorbed_fwd_workspace_bytes(S, h, d_c, d_nope, d_rope, d_v))
        return LAGA_ERR_WORKSPACE_TOO_SMALL;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    if ((rc = check_pointers({q, c_kv, k_pe, w_kv_b, out, lse, workspace})) != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    unsigned* status = reinterpret_cast<unsigned*>(base);
    const size_t lat_bytes = align_up(static_cast<size_t>(S) * h * kDc * 2, 1024);
    void* q_abs = base + kStatusBytes;
    void* o_lat = base + kStatusBytes + lat_bytes;
    if ((rc = zero_status(status, st)) != LAGA_OK) return rc;
    if ((rc = launch_q_absorb(q, w_kv_b, S, h, q_abs, status, st)) != LAGA_OK) return rc;
    if ((rc = launch_attn_absorbed(q, q_abs, c_kv, k_pe, S, h, softmax_scale, causal, o_lat, lse, status, st)) != LAGA_OK)
        return rc;
    return launch_v_project(o_lat, w_kv_b, S, h, out, status, st);
}

int laga_selftest_bounded_wait(void* status_word, unsigned budget_us, void* stream) {
    if (!status_word || budget_us < 1 || budget_us > 1000000) return LAGA_ERR_INVALID_ARG;
    int rc = check_device();
    if (rc != LAGA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((rc = zero_status_word(status_word, st)) != LAGA_OK) return rc;
    selftest_bounded_wait_kernel<<<1, 64, 0, st>>>(static_cast<unsigned*>(status_word),
                                                   static_cast<unsigned long long>(budget_us) * 1000ull);
    return launch_status();
}

int laga_profile_kernel(int kernel_id, void* const* start_events, void* const* stop_events, int n_pairs) {
    if (kernel_id < 0 || kernel_id >= LAGA_KERNEL_COUNT || n_pairs < 0) return LAGA_ERR_INVALID_ARG;
    if (n_pairs > 0 && (!start_events || !stop_events)) return LAGA_ERR_INVALID_ARG;
    for (int i = 0; i < n_pairs; ++i)
        if (!start_events[i] || !stop_events[i]) return LAGA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    ProfileSlot& slot = g_profile[kernel_id];
    slot.starts.clear();
    slot.stops.clear();
    slot.launches = 0;
    for (int i = 0; i < n_pairs; ++i) {
        slot.starts.push_back(static_cast<cudaEvent_t>(start_events[i]));
        slot.stops.push_back(static_cast<cudaEvent_t>(stop_events[i]));
    }
    return LAGA_OK;
}

int laga_query_kernel_clocks(const void* workspace, void* stream, double* sm_mhz, double* kernel_ms) {
    if (!workspace || !sm_mhz || !kernel_ms) return LAGA_ERR_INVALID_ARG;
    ClockProbe probes[4];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(probes, static_cast<const uint8_t*>(workspace) + kProbeOffsetBytes, sizeof(probes),
                        cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return LAGA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LAGA_ERR_CUDA;
    for (int k = 0; k < LAGA_KERNEL_COUNT; ++k) sm_mhz[k] = kernel_ms[k] = 0.0;
    const int ids[4] = {LAGA_KERNEL_ATTN_FWD, LAGA_KERNEL_ATTN_BWD_DKV, LAGA_KERNEL_ATTN_BWD_DQ, LAGA_KERNEL_ATTN_BWD_FUSED};
    for (int i = 0; i < 4; ++i) {
        const ClockProbe& p = probes[i];
        if (p.ns_end <= p.ns_begin || p.cycles_end <= p.cycles_begin) continue;   // that kernel has not run on this workspace
        const double ns = static_cast<double>(p.ns_end - p.ns_begin);
        sm_mhz[ids[i]] = static_cast<double>(p.cycles_end - p.cycles_begin) / ns * 1e3;
        kernel_ms[ids[i]] = ns * 1e-6;
    }
    return LAGA_OK;
}

int laga_query_status(const void* workspace, void* stream, unsigned* detail) {
    if (!workspace) return LAGA_ERR_INVALID_ARG;
    unsigned word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return LAGA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LAGA_ERR_CUDA;
    if (detail) *detail = word;
    if (word == 0) return LAGA_OK;
    if ((word & 0xff000000u) == kStatusTimeout) return LAGA_ERR_DEVICE_TIMEOUT;
    if ((word & 0xff000000u) == kStatusCheck) return LAGA_ERR_DEVICE_CHECK;
    return LAGA_ERR_CUDA;
}

}  // extern "C"
