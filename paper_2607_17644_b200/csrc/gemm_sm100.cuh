// Dense bf16 x bf16 -> fp32 GEMM on tcgen05 tensor cores with TMEM accumulators, fed by TMA.
// Used for the three contractions with the latent (Algorithm 1 step 4 and its two transposes in
// the backward of Section 5.2):
//     KV    [S, N]   = c_kv [S, d_c] . W [d_c, N]          A K-major,  B MN-major, bf16 out
//     dc_kv [S, d_c] = dKV  [S, N]   . W^T                 A K-major,  B K-major,  bf16 out
//     dW    [d_c, N] = c_kv^T . dKV                        A MN-major, B MN-major, fp32 atomic out (split-K)
// and, batched over the heads of the shard, for the two projections of the absorbed form (Section 3.2):
//     q_abs [S, h, d_c]  = q_nope [S, h, d_n] . W_uk[h]^T  A K-major,  B K-major,  bf16 out
//     out   [S, h, d_v]  = o_lat  [S, h, d_c] . W_uv[h]    A K-major,  B MN-major, bf16 out
// (a batch shifts the operands' innermost TMA coordinate and the output's column by a fixed step).
//
// Persistent: one CTA per SM walks the 128 x BN output tiles (n fastest, so neighbouring CTAs share
// the A tile through L2).  Warp 0 issues TMA loads, warp 1 issues the MMAs, warps 2..5 drain the
// accumulator from TMEM (each warp owns the 32 TMEM lanes its warp-id-mod-4 selects).  There are two
// accumulators of BN columns, so the epilogue of one tile runs under the main loop of the next.
// Operand tiles are 64 K-elements deep, 128-byte swizzled, STAGES deep.
#pragma once
#include "sm100_ptx.cuh"

namespace laga {

struct GemmArgs {
    int M, N, K;          // problem size; M may be ragged; N % 8 == 0 (CTA-pair kernel: any such N; one-CTA kernel: N % BN == 0);
                          // the K tail is zero-filled by TMA
    int k_tiles_per_split;
    int n_splits;         // split-K factor (1 unless EPI_ATOMIC_F32)
    void* C;              // bf16 [M, ldc] (EPI_BF16) or fp32 [M, ldc] (EPI_ATOMIC_F32)
    int ldc;
    unsigned int* status;
    float4* zero_begin;   // optional: zero_count float4 elements cleared by this launch before it starts
    size_t zero_count;    // (the buffer the NEXT kernel accumulates into: saves a separate memset)
    int batches;          // >= 1; batch b adds b * a_step / b_step to the operands' innermost (contiguous)
    int a_step, b_step;   // TMA coordinate and b * c_step to the output column
    int c_step;
};

enum { EPI_BF16 = 0, EPI_ATOMIC_F32 = 1 };

template <int BN, int STAGES>
struct GemmSmem {
    static constexpr int kABytes = 128 * 64 * 2;
    static constexpr int kBBytes = BN * 64 * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kBarrierOffset = STAGES * kStageBytes;
    static constexpr int kTotalBytes = kBarrierOffset + 256 + 1024;   // + alignment slack
};

template <int BN, int STAGES, bool A_MN, bool B_MN, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const GemmArgs args) {
    using L = GemmSmem<BN, STAGES>;
    static_assert(2 * BN <= 512, "two accumulators must fit in TMEM");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::kBarrierOffset);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_full = empty_bar + STAGES;   // [2]
    uint64_t* acc_empty = acc_full + 2;        // [2]
    uint64_t* quiesce_bar = acc_empty + 2;     // abort path only: the MMA lane's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(quiesce_bar + 1);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_n = args.N / BN;
    const int tiles_m = (args.M + 127) / 128;
    const int tiles_per_batch = tiles_n * tiles_m * args.n_splits;
    const int total_tiles = tiles_per_batch * args.batches;
    const int total_k_tiles = (args.K + 63) / 64;
    constexpr uint32_t kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 128); }
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();          // global memory from here on
    for (size_t z = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; z < args.zero_count;
         z += static_cast<size_t>(gridDim.x) * blockDim.x)
        args.zero_begin[z] = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint32_t tmem_base = *tmem_slot;

    auto k_range = [&](int split, int& kt_begin, int& n_kt) {
        kt_begin = split * args.k_tiles_per_split;
        const int kt_end = min(total_k_tiles, kt_begin + args.k_tiles_per_split);
        n_kt = max(0, kt_end - kt_begin);
    };

    if (warp == 0) {
        if (elect_one()) {
            uint32_t kc = 0;   // running k-iteration count: stage = kc % STAGES, phase = (kc / STAGES) & 1
            bool ok = true;
            ArmedBarriers armed(full_bar);
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const int batch = t / tiles_per_batch, tb = t - batch * tiles_per_batch;
                const int n0 = (tb % tiles_n) * BN, m0 = ((tb / tiles_n) % tiles_m) * 128;
                const int a_off = batch * args.a_step, b_off = batch * args.b_step;
                int kt_begin, n_kt;
                k_range(tb / (tiles_n * tiles_m), kt_begin, n_kt);
                for (int i = 0; i < n_kt; ++i, ++kc) {
                    const int s = kc % STAGES;
                    ok = mbar_wait(&empty_bar[s], ((kc / STAGES) & 1) ^ 1, abort_flag, args.status, 0x100);
                    if (!ok) break;
                    uint8_t* sa = smem + s * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    mbar_arrive_expect_tx(&full_bar[s], L::kStageBytes);
                    armed.arm(&full_bar[s], (kc / STAGES) & 1);
                    const int k0 = (kt_begin + i) * 64;
                    if (A_MN) {   // global A is [K rows, M contiguous]: two slabs of 64 K-rows x 64 M
                        tma_load_2d_chk(args.status, sa, &tmap_a, &full_bar[s], a_off + m0, k0);
                        tma_load_2d_chk(args.status, sa + 8192, &tmap_a, &full_bar[s], a_off + m0 + 64, k0);
                    } else {      // global A is [M rows, K contiguous]: one slab of 128 rows x 64 K
                        tma_load_2d_chk(args.status, sa, &tmap_a, &full_bar[s], a_off + k0, m0);
                    }
                    if (B_MN) {
                        for (int j = 0; j < BN / 64; ++j)
                            tma_load_2d_chk(args.status, sb + j * 8192, &tmap_b, &full_bar[s], b_off + n0 + j * 64, k0);
                    } else {
                        tma_load_2d_chk(args.status, sb, &tmap_b, &full_bar[s], b_off + k0, n0);
                    }
                }
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(128, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
            uint32_t kc = 0, it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                int kt_begin, n_kt;
                k_range((t % tiles_per_batch) / (tiles_n * tiles_m), kt_begin, n_kt);
                const uint32_t buf = it & 1;
                ok = mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, args.status, 0x201);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tmem_acc = tmem_base + buf * BN;
                for (int i = 0; i < n_kt; ++i, ++kc) {
                    const int s = kc % STAGES;
                    ok = mbar_wait(&full_bar[s], (kc / STAGES) & 1, abort_flag, args.status, 0x200);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(smem + s * L::kStageBytes);
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t da = A_MN ? desc_mn_major(sa + k * 2048, 8192) : desc_k_major(sa + k * 32);
                        const uint64_t db = B_MN ? desc_mn_major(sb + k * 2048, 8192) : desc_k_major(sb + k * 32);
                        mma_ss(tmem_acc, da, db, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(&empty_bar[s]);
                }
                if (ok) mma_commit(&acc_full[buf]);
            }
            if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        // Epilogue: TMEM lane = output row within the tile, TMEM column = output column.
        const int quarter = warp & 3;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        uint32_t it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
            const int batch = t / tiles_per_batch, tb = t - batch * tiles_per_batch;
            const int n0 = batch * args.c_step + (tb % tiles_n) * BN, m0 = ((tb / tiles_n) % tiles_m) * 128;
            int kt_begin, n_kt;
            k_range(tb / (tiles_n * tiles_m), kt_begin, n_kt);
            const uint32_t buf = it & 1;
            const int row = m0 + quarter * 32 + lane;
            ok = mbar_wait_warp(&acc_full[buf], (it >> 1) & 1, abort_flag, args.status, 0x300);
            if (!ok) break;
            tc_fence_after_sync();
            if (n_kt > 0) {
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld_x32(tmem_base + lane_addr + buf * BN + c * 32, r);
                    tmem_ld_wait();
                    if (row < args.M) {
                        if (EPI == EPI_BF16) {
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(args.C) +
                                                 static_cast<size_t>(row) * args.ldc + n0 + c * 32;
                            uint4* dst4 = reinterpret_cast<uint4*>(dst);
                            if (!device_check(aligned16_dev(dst) && n0 + c * 32 + 32 <= args.ldc, args.status, 0xE10000u | c)) continue;
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                uint4 o;
                                o.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                                o.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                                o.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                                o.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                                dst4[v] = o;
                            }
                        } else {
                            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.C) +
                                                                    static_cast<size_t>(row) * args.ldc + n0 + c * 32);
                            if (!device_check(aligned16_dev(dst) && n0 + c * 32 + 32 <= args.ldc, args.status, 0xE20000u | c)) continue;
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                atomicAdd(dst + v, make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                                               __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3])));
                        }
                    }
                }
            }
            __syncwarp();
            tc_fence_before_sync();
            mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, kTmemCols); }
}

// ------------------------------------------------------------------------------------------------
// The same GEMM on CTA PAIRS (cluster of two, tcgen05 cta_group::2): a pair owns 256 x BN output tiles,
// each CTA holds its own 128 rows of A and half of the BN columns of B, so a CTA fills (and the MMAs read)
// 16 + 16 KB per 64-deep k-stage instead of 16 + 32 KB for the same 128 x BN outputs per CTA.  With K = 512
// the one-CTA kernel is bound by those fills (it moves 384 KB from L2 for every 33 MFLOP tile).
// Roles per CTA as above; only the even CTA's warp 1 issues MMAs and commits, to barriers in both CTAs.
// The full barriers live in the even CTA and count the bytes of both CTAs' loads; the odd CTA's epilogue
// warps release the accumulator buffer with arrivals on the even CTA's barrier.
template <int BN, int STAGES>
struct GemmPairSmem {
    static constexpr int kABytes = 128 * 64 * 2;
    static constexpr int kBBytes = (BN / 2) * 64 * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStoreOffset = STAGES * kStageBytes;     // bf16 epilogue: 4 warps x 2 buffers x (32 rows x 128 B)
    static constexpr int kStoreBytes = 4 * 2 * 4096;
    static constexpr int kBarrierOffset = kStoreOffset + kStoreBytes;
    static constexpr int kTotalBytes = kBarrierOffset + 256;
};

// bf16 epilogue: every lane owns one output row; writing it straight to global memory costs one wavefront
// per lane and 16-byte store (the rows are kilobytes apart), which for a 128 x 256 tile is as many load/store
// cycles as the tile's MMAs take.  Instead each warp packs 64 columns of its 32 rows into a 128-byte-swizzled
// 4 KB box in shared memory (4-way bank conflicts instead of 32 wavefronts) and one lane hands the box to TMA
// (`tmap_c`: the output as [rows, ldc] bf16, box 64 x 32); two boxes per warp alternate so that packing the
// next one overlaps the store of the last.  TMA clips rows past M.
template <int BN, int STAGES, bool A_MN, bool B_MN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 1)
gemm_pair_sm100_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                       const __grid_constant__ CUtensorMap tmap_c, const GemmArgs args) {
    using L = GemmPairSmem<BN, STAGES>;
    static_assert(2 * BN <= 512 && BN % 128 == 0, "two accumulators must fit in TMEM; each CTA holds whole 64-column slabs");
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::kBarrierOffset);   // used in the even CTA only
    uint64_t* empty_bar = full_bar + STAGES;   // both CTAs: the stage's MMAs have completed
    uint64_t* acc_full = empty_bar + STAGES;   // [2] both CTAs
    uint64_t* acc_empty = acc_full + 2;        // [2] even CTA: 256 arrivals (both CTAs' epilogue threads)
    uint64_t* quiesce_bar = acc_empty + 2;     // abort path only: the MMA lane's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(quiesce_bar + 1);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int tiles_n = (args.N + BN - 1) / BN;   // the last column tile may be ragged: loads past N are zero fill, stores are clipped
    const int tiles_m = (args.M + 255) / 256;
    const int tiles_per_batch = tiles_n * tiles_m * args.n_splits;
    const int total_tiles = tiles_per_batch * args.batches;
    const int total_k_tiles = (args.K + 63) / 64;
    constexpr uint32_t kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 256); }
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
        if ((smem_u32(smem) & 1023u) != 0u) {
            abort_flag->value = 1;
        }
    }
    if (warp == 1) { tmem_alloc_pair(tmem_slot, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();            // the peer's barriers exist before anything can arrive on them
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();    // global memory from here on
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD4u);   // set-up found the shared memory misaligned
    for (size_t z = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; z < args.zero_count;
         z += static_cast<size_t>(gridDim.x) * blockDim.x)
        args.zero_begin[z] = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint32_t tmem_base = *tmem_slot;
    const bool run = abort_flag->value == 0u;   // (the layout is the same in both CTAs: they agree)

    auto k_range = [&](int split, int& kt_begin, int& n_kt) {
        kt_begin = split * args.k_tiles_per_split;
        const int kt_end = min(total_k_tiles, kt_begin + args.k_tiles_per_split);
        n_kt = max(0, kt_end - kt_begin);
    };

    if (!run) {
        // fall through to the common exit
    } else if (warp == 0) {
        if (elect_one()) {
            uint32_t kc = 0;
            bool ok = true;
            ArmedBarriers armed(full_bar);
            for (int t = pair; t < total_tiles && ok; t += n_pairs) {
                const int batch = t / tiles_per_batch, tb = t - batch * tiles_per_batch;
                const int n0 = (tb % tiles_n) * BN + static_cast<int>(rank) * (BN / 2);
                const int m0 = ((tb / tiles_n) % tiles_m) * 256 + static_cast<int>(rank) * 128;
                const int a_off = batch * args.a_step, b_off = batch * args.b_step;
                int kt_begin, n_kt;
                k_range(tb / (tiles_n * tiles_m), kt_begin, n_kt);
                for (int i = 0; i < n_kt; ++i, ++kc) {
                    const int s = kc % STAGES;
                    ok = mbar_wait(&empty_bar[s], ((kc / STAGES) & 1) ^ 1, abort_flag, args.status, 0x110);
                    if (!ok) break;
                    uint8_t* sa = smem + s * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    if (rank == 0) { mbar_arrive_expect_tx(&full_bar[s], 2 * L::kStageBytes); armed.arm(&full_bar[s], (kc / STAGES) & 1); }   // both CTAs' bytes
                    const uint32_t bar = cluster_map(&full_bar[s], 0);
                    const int k0 = (kt_begin + i) * 64;
                    if (A_MN) {
                        tma_load_2d_pair_chk(args.status, sa, &tmap_a, bar, a_off + m0, k0);
                        tma_load_2d_pair_chk(args.status, sa + 8192, &tmap_a, bar, a_off + m0 + 64, k0);
                    } else {
                        tma_load_2d_pair_chk(args.status, sa, &tmap_a, bar, a_off + k0, m0);
                    }
                    if (B_MN) {
                        for (int j = 0; j < BN / 128; ++j)
                            tma_load_2d_pair_chk(args.status, sb + j * 8192, &tmap_b, bar, b_off + n0 + j * 64, k0);
                    } else {
                        tma_load_2d_pair_chk(args.status, sb, &tmap_b, bar, b_off + k0, n0);
                    }
                }
            }
            // (the final cluster barrier keeps the odd CTA's shared memory alive until the even CTA has seen
            // these barriers complete or given up on them)
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 1) {
        if (rank == 0 && elect_one()) {
            constexpr uint32_t idesc = make_idesc_bf16(256, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
            uint32_t kc = 0, it = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += n_pairs, ++it) {
                int kt_begin, n_kt;
                k_range((t % tiles_per_batch) / (tiles_n * tiles_m), kt_begin, n_kt);
                const uint32_t buf = it & 1;
                ok = mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, args.status, 0x211);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tmem_acc = tmem_base + buf * BN;
                for (int i = 0; i < n_kt; ++i, ++kc) {
                    const int s = kc % STAGES;
                    ok = mbar_wait(&full_bar[s], (kc / STAGES) & 1, abort_flag, args.status, 0x210);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(smem + s * L::kStageBytes);
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t da = A_MN ? desc_mn_major(sa + k * 2048, 8192) : desc_k_major(sa + k * 32);
                        const uint64_t db = B_MN ? desc_mn_major(sb + k * 2048, 8192) : desc_k_major(sb + k * 32);
                        mma_ss_pair(tmem_acc, da, db, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit_pair(&empty_bar[s], 3);
                }
                if (ok) mma_commit_pair(&acc_full[buf], 3);
            }
            if (abort_flag->value != 0u) { mma_commit_pair(quiesce_bar, 1); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        const int quarter = warp & 3;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        const uint32_t acc_empty_leader[2] = {cluster_map(&acc_empty[0], 0), cluster_map(&acc_empty[1], 0)};
        uint8_t* store_base = smem + L::kStoreOffset + quarter * 2 * 4096;   // this warp's two output boxes
        uint32_t boxes = 0;
        uint32_t it = 0;
        bool ok = true;
        for (int t = pair; t < total_tiles && ok; t += n_pairs, ++it) {
            const int batch = t / tiles_per_batch, tb = t - batch * tiles_per_batch;
            const int n0 = batch * args.c_step + (tb % tiles_n) * BN;
            const int m0 = ((tb / tiles_n) % tiles_m) * 256 + static_cast<int>(rank) * 128;
            int kt_begin, n_kt;
            k_range(tb / (tiles_n * tiles_m), kt_begin, n_kt);
            const uint32_t buf = it & 1;
            const int row = m0 + quarter * 32 + lane;
            ok = mbar_wait_warp(&acc_full[buf], (it >> 1) & 1, abort_flag, args.status, 0x310);
            if (!ok) break;
            tc_fence_after_sync();
            if (n_kt > 0) {
                if (EPI == EPI_BF16) {
#pragma unroll 1
                    for (int c = 0; c < BN / 64; ++c, ++boxes) {
                        if ((tb % tiles_n) * BN + c * 64 >= args.N) break;   // past the last column (ragged N); TMA clips a partial box
                        uint32_t r[64];
                        __syncwarp();
                        tmem_ld_x32(tmem_base + lane_addr + buf * BN + c * 64, r);
                        tmem_ld_x32(tmem_base + lane_addr + buf * BN + c * 64 + 32, r + 32);
                        tmem_ld_wait();
                        uint8_t* box = store_base + (boxes & 1u) * 4096;
                        if (lane == 0) tma_store_wait_read<1>();       // the box used two stores ago has been read
                        __syncwarp();
#pragma unroll
                        for (int v = 0; v < 8; ++v) {                   // 16-byte chunk v of this lane's 128-byte row
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                            o.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                            o.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                            o.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                            *reinterpret_cast<uint4*>(box + lane * 128 + ((v ^ (lane & 7)) << 4)) = o;
                        }
                        fence_async_shared();
                        __syncwarp();
                        if (lane == 0 && device_check(((n0 + c * 64) & 7) == 0 && n0 + c * 64 < args.ldc, args.status, 0xE70000u | c)) {
                            tma_store_2d(&tmap_c, box, n0 + c * 64, m0 + quarter * 32);
                            tma_store_commit();
                        }
                    }
                } else {
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        const int col = (tb % tiles_n) * BN + c * 32;       // column within this batch's N
                        if (col >= args.N) break;                           // ragged N: nothing beyond the last column
                        uint32_t r[32];
                        __syncwarp();
                        tmem_ld_x32(tmem_base + lane_addr + buf * BN + c * 32, r);
                        tmem_ld_wait();
                        if (row < args.M) {
                            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.C) +
                                                                    static_cast<size_t>(row) * args.ldc + n0 + c * 32);
                            if (!device_check(aligned16_dev(dst) && n0 + c * 32 < args.ldc, args.status, 0xE20000u | c)) continue;
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                if (col + v * 4 + 4 <= args.N)
                                    atomicAdd(dst + v, make_float4(__uint_as_float(r[v * 4]), __uint_as_float(r[v * 4 + 1]),
                                                                   __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3])));
                        }
                    }
                }
            }
            __syncwarp();
            tc_fence_before_sync();
            mbar_arrive_cluster(acc_empty_leader[buf]);
        }
        if (EPI == EPI_BF16 && lane == 0) tma_store_wait_all();   // the stores read shared memory until they complete
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();            // neither CTA frees TMEM or leaves while the peer may still use it or its barriers
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc_pair(tmem_base, kTmemCols); }
}

}  // namespace laga
