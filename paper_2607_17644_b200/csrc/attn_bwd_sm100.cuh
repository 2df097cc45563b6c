// Backward of Algorithm 1 step 5 (Section 5.2: the chain rule through the softmax attention) for
// the DeepSeek-V3 head geometry, as two persistent tcgen05 kernels that recompute P from the saved LSE:
//
//   attn_bwd_dkv  one (128-key tile, head) item at a time per CTA, sweeping the 128-row query tiles that
//                 attend to it: S^T = K Q^T, dP^T = V dO^T, P^T = exp(scale S^T - LSE),
//                 dS^T = P^T (dP^T - delta), dV += P^T dO, dK += dS^T Q (dK 192 wide: 128 nope columns +
//                 64 rope columns).  TMEM lanes are keys, so LSE and delta are per-column vectors staged
//                 in shared memory.
//   attn_bwd_dq   one (128-query tile, head) item at a time per CTA, sweeping 128-key tiles:
//                 S = Q K^T, dP = dO V^T, dS = P (dP - delta), dQ += dS K.  TMEM lanes are queries.
//
// Both read K_nope / V from the recomputed bf16 up-projection KV[S, h*256] and the shared rope band
// from k_pe[S, 64]; both keep every accumulator in TMEM and never materialise S x S.  With packed
// variable-length sequences (work_sched.cuh: SeqTile) an item is a tile of one sequence and every index
// below is relative to that sequence.
//
// Roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 and 6..9 two consumer
// warpgroups (every thread owns one TMEM lane; the groups split a tile's 128 columns).  P^T / dS^T (dkv)
// and dS (dq) never touch shared memory: the consumers write them back to TMEM as packed bf16 and the
// accumulating MMAs read their A operand from there.  Scratch columns are reused by an MMA that the same
// thread issues after the MMAs that read them; the tensor pipe runs one thread's MMAs in order, so that
// reuse needs no barrier.
//   dkv: dK (192) + dV (128) leave 192 TMEM columns: X (128, fp32: S^T then dP^T) and Y (64, bf16: P^T then
//        dS^T) for ONE 128-wide tile, so that every MMA is at least 128 wide (a 64-wide N costs 48 cycles
//        per MMA against 32 ideal and re-reads its A tile for half the work).
//   dq:  128-key tiles, all MMAs 128 wide.  dO (the A operand of dP) lives in TMEM, which frees shared
//        memory for a third K stage.
#pragma once
#include "attn_fwd_sm100.cuh"
#include "sm100_ptx.cuh"
#include "work_sched.cuh"

namespace laga {

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gmem_src)), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// ---- delta and transposed softmax statistics ---------------------------------------------------
// delta[s,i] = sum_d dO[s,i,d] O[s,i,d].  Written head-major and padded: stat_l2[i][s] = LSE*log2(e),
// stat_delta[i][s] = delta for s < S; for S <= s < S_pad the entries are (+inf, 0) so that query rows
// past the end of the sequence produce P = 0.  (S here counts the rows of out / dout / lse; S_pad the
// padded positions, which for packed sequences exceed it by each sequence's own padding.)
// Eight lanes per (row, head): each lane reads 16 channels of O and dO as two 16-byte loads apiece.
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                 const float* __restrict__ lse, int S, int h, int S_pad, float* __restrict__ stat_l2,
                 float* __restrict__ stat_delta, float4* __restrict__ zero_begin, size_t zero_count,
                 const int2* __restrict__ seqs, int n_seqs) {
    // This kernel depends on nothing the kernel launched before it in the same call produces (that is the
    // recomputed up-projection: it writes K/V, this reads out / dout / lse and writes the statistics and the
    // rope-gradient accumulator), so it does not wait for it before working: launched with programmatic stream
    // serialization it runs BESIDE the up-projection (bound by HBM, the other by the tensor pipe).  It waits at
    // its END instead, so that its own completion still implies the completion of everything before it -- the
    // kernels after it rely on that.
    grid_launch_dependents();
    // Also clears the fp32 buffer the dK/dV kernel accumulates the rope-column key gradients into
    // (zero_count float4 elements): one launch less than a separate memset.
    for (size_t z = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; z < zero_count;
         z += static_cast<size_t>(gridDim.x) * blockDim.x)
        zero_begin[z] = make_float4(0.f, 0.f, 0.f, 0.f);
    const long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 3;   // (padded row, head) pair
    const int sub = threadIdx.x & 7;
    const bool live = item < static_cast<long long>(S_pad) * h;
    const int s = live ? static_cast<int>(item / h) : 0, i = live ? static_cast<int>(item % h) : 0;
    // Packed sequences (seqs != nullptr): entry k is (first row, first padded position) of sequence k, entry
    // n_seqs closes the list; every sequence is padded to a multiple of 128 positions of its own.  Padded
    // position s belongs to the last sequence whose padded start is <= s.
    int row = s;
    bool valid = s < S;
    if (seqs != nullptr) {
        int lo = 0, hi = n_seqs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (seqs[mid].y <= s) lo = mid; else hi = mid - 1;
        }
        const int local = s - seqs[lo].y;
        row = seqs[lo].x + local;
        valid = row < seqs[lo + 1].x;
    }
    float acc = 0.f;
    if (live && valid) {
        const size_t base = (static_cast<size_t>(row) * h + i) * 128 + sub * 16;
        const uint4 a0 = *reinterpret_cast<const uint4*>(out + base), a1 = *reinterpret_cast<const uint4*>(out + base + 8);
        const uint4 b0 = *reinterpret_cast<const uint4*>(dout + base), b1 = *reinterpret_cast<const uint4*>(dout + base + 8);
        const uint32_t aw[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        const uint32_t bw[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[k]));
            const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[k]));
            acc = fmaf(x.x, y.x, acc);
            acc = fmaf(x.y, y.y, acc);
        }
    }
#pragma unroll
    for (int off = 4; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (live && sub == 0) {
        stat_l2[static_cast<size_t>(i) * S_pad + s] = valid ? lse[static_cast<size_t>(row) * h + i] * 1.4426950408889634f : INFINITY;
        stat_delta[static_cast<size_t>(i) * S_pad + s] = valid ? acc : 0.f;
    }
    grid_dependency_wait();
}

// dk_pe[t, r] is the sum over heads of the rope-column key gradients (Section 5.3: the rope band is
// shared by every head, so its gradient is the sum over the head shard).  The dK/dV kernel adds each
// head's columns into an fp32 accumulator with atomics; this kernel rounds the sums to bf16.
__global__ void __launch_bounds__(256)
bwd_dkpe_convert_kernel(const float* __restrict__ dkpe_acc, int S, __nv_bfloat16* __restrict__ dk_pe) {
    // Launched behind the dQ kernel, whose output it does not touch: what it reads is complete once the dQ
    // kernel's CTAs have passed THEIR dependency wait (they signal their dependents only after it), so it starts
    // beside them and, like the delta kernel, waits at its end.  The sums were written by another grid's atomics:
    // they are read past L1.
    grid_launch_dependents();
    const size_t idx = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
    if (idx < static_cast<size_t>(S) * 64) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(dkpe_acc + idx));
        uint2 o;
        o.x = pack_bf16x2(v.x, v.y);
        o.y = pack_bf16x2(v.z, v.w);
        *reinterpret_cast<uint2*>(dk_pe + idx) = o;
    }
    grid_dependency_wait();
}

// Deterministic alternative to the atomics: sum the per-head buffers in head order.
__global__ void __launch_bounds__(256)
bwd_dkpe_reduce_kernel(const float* __restrict__ dk_rope, int S, int h, __nv_bfloat16* __restrict__ dk_pe) {
    grid_launch_dependents();
    grid_dependency_wait();
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t n = static_cast<size_t>(S) * 64;
    if (idx >= n) return;
    float acc = 0.f;
    for (int i = 0; i < h; ++i) acc += dk_rope[static_cast<size_t>(i) * n + idx];
    dk_pe[idx] = __float2bfloat16_rn(acc);
}

constexpr int kBwdThreads = 320;

// ================================================================================================
// dK / dV kernel
// ================================================================================================
struct AttnBwdDkvArgs {
    int S, h, S_pad;
    float scale_log2, scale;
    const float* stat_l2;      // [h][S_pad]
    const float* stat_delta;   // [h][S_pad]
    __nv_bfloat16* dkv;        // [S, h*256]: per head dK_nope (128) then dV (128)
    float* dkpe_acc;           // [S][64] fp32, zero when the kernel starts; every head's CTA adds into it
    float* dk_rope_per_head;   // deterministic mode: [h][S][64] fp32 written per head (then summed in a fixed
                               // order by bwd_dkpe_reduce_kernel); nullptr selects the atomic path
    unsigned int* status;
    WorkSchedule sched;        // items = (128-key tile, head); rank 0 = key tile 0 (every query attends to it)
    ClockProbe* clock_probe;   // may be nullptr
};

struct AttnBwdDkvSmem {
    static constexpr int kSlab = 128 * 128;                    // 128 rows x 128 B
    static constexpr int kQStages = 2;
    static constexpr int kK = 0;                               // 3 slabs: K_nope (2), rope band (1)
    static constexpr int kV = kK + 3 * kSlab;                  // 2 slabs
    static constexpr int kQ = kV + 2 * kSlab;                  // kQStages x 3 slabs
    static constexpr int kDo = kQ + kQStages * 3 * kSlab;      // 1 stage x 2 slabs
    static constexpr int kStat = kDo + 2 * kSlab;              // per Q stage: 128 l2 + 128 delta floats
    static constexpr int kBar = kStat + kQStages * 1024;
    static constexpr int kTotalBytes = kBar + 512;
};
static_assert(AttnBwdDkvSmem::kTotalBytes <= 232448, "dkv kernel exceeds the 227 KB of shared memory per CTA");

// Persistent: one CTA per SM takes (key tile, head) items from the work counter.  Per item the 128-key
// K/V tile is stationary and the 128-row query tiles that attend to it stream through.  Every MMA is
// 128 wide or wider: a 64-wide tcgen05.mma re-reads its 4 KB A tile for half the work and costs 48
// clocks against 32, and this kernel is bound by the shared-memory port as much as by the tensor pipe.
// TMEM: X (128 columns, fp32) holds S^T and then dP^T of the tile; Y (64 columns, packed bf16) holds
// P^T and then dS^T, the A operands of the two accumulating MMAs; dK (192) and dV (128) fill the rest.
//     ... dV(j-1) | S^T(j) | dK(j-1) | dP^T(j) | dV(j) | S^T(j+1) | ...
// S^T(j) is issued as soon as the consumers have read dP^T(j-1) out of X, so the exponentials of tile j
// run under dK(j-1) and dP^T(j); dS^T(j-1) is computed under dV(j-1) and S^T(j).  The two consumer
// warpgroups split each tile's query columns (64 each).
//
// kRebuild (LAGA_FLAG_FUSED_KV_REBUILD): the up-projection of Algorithm 1 step 4 is fused into this kernel's item
// prologue instead of being recomputed by a GEMM launch of its own.  The item's K_nope / V tile
// [128 keys x 256] = c_kv[128 keys x 512] . W_kv_b[512 x 256 of the head] is built by 32 MMAs (N = 256) into the
// accumulator columns that dK / dV will occupy (they are free between items), from eight 64-deep chunks that the
// producer streams through the Q stages (one chunk = one c_kv slab + a 64 x 256 block of W = exactly one stage;
// eight chunks are four turns of the two-stage ring, so the Q tiles' stage and phase numbering is unchanged).  The
// consumers round the tile to bf16 and write it into the K and V operand slabs in the swizzled layout a TMA load
// would have produced; one of them also stores the four slabs to the K/V workspace, which the dQ kernel reads
// afterwards.  Only the shared rope band still comes from memory.  The key-stationary loop is the one place where
// this fusion costs no extra arithmetic (each K/V tile is built once).
template <bool kCausal, bool kRebuild = false>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_dkv_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                          const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                          const __grid_constant__ CUtensorMap tmap_ckv, const __grid_constant__ CUtensorMap tmap_w,
                          const AttnBwdDkvArgs args) {
    using L = AttnBwdDkvSmem;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* kv_full = bars + 0;
    uint64_t* kv_empty = bars + 1;    // the item's last S^T / dP^T have read K and V
    uint64_t* q_full = bars + 2;      // [2]  Q tile and its statistics
    uint64_t* q_empty = bars + 4;     // [2]
    uint64_t* do_full = bars + 6;
    uint64_t* do_empty = bars + 7;
    uint64_t* st_full = bars + 8;     // S^T of the tile is in X
    uint64_t* st_read = bars + 9;     // both groups have loaded it: X may take dP^T
    uint64_t* dp_full = bars + 10;    // dP^T is in X
    uint64_t* dp_read = bars + 11;    // both groups have loaded it: X may take the next S^T
    uint64_t* p_full = bars + 12;     // P^T (bf16) is in Y
    uint64_t* dv_done = bars + 13;    // dV += P^T dO has read Y: it may take dS^T
    uint64_t* ds_full = bars + 14;    // dS^T (bf16) is in Y
    uint64_t* dk_done = bars + 15;    // dK += dS^T Q has read Y: it may take the next P^T
    uint64_t* acc_full = bars + 16;   // the item's dK / dV are complete
    uint64_t* acc_empty = bars + 17;  // both groups have drained them
    ItemRing ring{bars + 18, bars + 20, reinterpret_cast<volatile int*>(bars + 22)};
    uint64_t* quiesce_bar = bars + 23;   // abort path only: the MMA lane's last commit
    uint64_t* rb_full = bars + 24;       // kRebuild: the item's K_nope / V tile is in TMEM (fp32)
    uint64_t* kv_built = bars + 25;      // kRebuild: both groups have written it to the operand slabs
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1); mbar_init(kv_empty, 1);
        mbar_init(rb_full, 1); mbar_init(kv_built, 256);
        if (kRebuild) { tma_prefetch_desc(&tmap_ckv); tma_prefetch_desc(&tmap_w); }
        for (int s = 0; s < L::kQStages; ++s) { mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1); }
        mbar_init(do_full, 1); mbar_init(do_empty, 1);
        mbar_init(st_full, 1); mbar_init(st_read, 256); mbar_init(dp_full, 1); mbar_init(dp_read, 256);
        mbar_init(p_full, 256); mbar_init(dv_done, 1); mbar_init(ds_full, 256); mbar_init(dk_done, 1);
        mbar_init(acc_full, 1); mbar_init(acc_empty, 256);
        for (int s = 0; s < 2; ++s) { mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], 9); }
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_do);
        tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
        if ((smem_u32(smem) & 1023u) != 0u) {   // the swizzled operand slabs need a 1024-byte aligned base
            abort_flag->value = 1;
        }
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();          // set-up above overlaps the previous kernel's tail; global memory from here on
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD0u);   // set-up found the shared memory misaligned
    clock_probe_begin(args.clock_probe);
    const uint32_t tmem_base = *tmem_slot;
    // columns: [0,128) X | [128,192) Y | [192,384) dK | [384,512) dV
    const uint32_t tmem_y = tmem_base + 128;
    const uint32_t tmem_dk = tmem_base + 192;
    const uint32_t tmem_dv = tmem_base + 384;
    // Indices are relative to the item's sequence (see SeqTile); `seq` carries its first row, its length
    // and its start in the padded statistics arrays.
    auto item_geometry = [&](int item, int& t0, int& head, int& j_begin, int& n_iter, SeqTile& seq) {
        int rank;
        decode_item(args.sched, item, rank, head);
        seq = seq_tile(args.sched, rank, args.S, false);   // key tile 0 has the most queries
        t0 = seq.tile * 128;
        j_begin = kCausal ? seq.tile : 0;
        n_iter = (seq.seq_len + 127) / 128 - j_begin;      // >= 1 because t0 < seq_len
    };

    if (abort_flag->value != 0u) {
        // misaligned shared memory: nothing was started, fall through to the common exit
    } else if (warp == 0) {
        if (elect_one()) {
            uint32_t T = 0;                      // running tile count of this CTA: ring positions and phases
            bool ok = true;
            ArmedBarriers armed(bars);
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_publish(ring, args.sched, n, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int t0, head, j_begin, n_iter;
                SeqTile seq;
                item_geometry(item, t0, head, j_begin, n_iter, seq);
                const int row_base = seq.seq_start;
                ok = mbar_wait(kv_empty, (n & 1u) ^ 1u, abort_flag, args.status, 0x41);
                if (!ok) break;
                if (!kRebuild) {
                    mbar_arrive_expect_tx(kv_full, 5 * L::kSlab);
                    armed.arm(kv_full, n & 1u);
                    tma_load_2d_chk(args.status, smem + L::kK, &tmap_kv, kv_full, head * 256, row_base + t0);
                    tma_load_2d_chk(args.status, smem + L::kK + L::kSlab, &tmap_kv, kv_full, head * 256 + 64, row_base + t0);
                    tma_load_2d_chk(args.status, smem + L::kK + 2 * L::kSlab, &tmap_kpe, kv_full, 0, row_base + t0);
                    tma_load_2d_chk(args.status, smem + L::kV, &tmap_kv, kv_full, head * 256 + 128, row_base + t0);
                    tma_load_2d_chk(args.status, smem + L::kV + L::kSlab, &tmap_kv, kv_full, head * 256 + 192, row_base + t0);
                } else {
                    // only the rope band is loaded; K_nope and V are built from eight chunks of the latent and the
                    // head's weight block, streamed through the Q stages ahead of the item's Q tiles (chunk c takes
                    // the ring position of tile T + c: eight positions are whole turns of the ring and of its phases)
                    mbar_arrive_expect_tx(kv_full, L::kSlab);
                    armed.arm(kv_full, n & 1u);
                    tma_load_2d_chk(args.status, smem + L::kK + 2 * L::kSlab, &tmap_kpe, kv_full, 0, row_base + t0);
                    for (uint32_t c = 0; c < 8u && ok; ++c) {
                        const uint32_t Tc = T + c, sq = Tc % L::kQStages;
                        ok = mbar_wait(&q_empty[sq], ((Tc / L::kQStages) & 1u) ^ 1u, abort_flag, args.status, 0x43);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&q_full[sq], 3 * L::kSlab);
                        armed.arm(&q_full[sq], (Tc / L::kQStages) & 1u);
                        uint8_t* dst = smem + L::kQ + sq * 3 * L::kSlab;
                        tma_load_2d_chk(args.status, dst, &tmap_ckv, &q_full[sq], static_cast<int>(c) * 64, row_base + t0);
                        for (int b = 0; b < 4; ++b)     // 64 latent rows x 64 columns each: 8 KB boxes
                            tma_load_2d(dst + L::kSlab + b * 8192, &tmap_w, &q_full[sq], head * 256 + b * 64, static_cast<int>(c) * 64);
                    }
                    if (!ok) break;
                }
                for (int j = 0; j < n_iter; ++j, ++T) {
                    const uint32_t sq = T % L::kQStages;
                    const int q0 = (j_begin + j) * 128;
                    ok = mbar_wait(&q_empty[sq], ((T / L::kQStages) & 1u) ^ 1u, abort_flag, args.status, 0x40);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&q_full[sq], 3 * L::kSlab + 1024);
                    armed.arm(&q_full[sq], (T / L::kQStages) & 1u);
                    uint8_t* dst_q = smem + L::kQ + sq * 3 * L::kSlab;
                    for (int c = 0; c < 3; ++c)
                        tma_load_2d_chk(args.status, dst_q + c * L::kSlab, &tmap_q, &q_full[sq], head * 192 + c * 64, row_base + q0);
                    float* stat = reinterpret_cast<float*>(smem + L::kStat + sq * 1024);
                    bulk_load_1d(stat, args.stat_l2 + static_cast<size_t>(head) * args.S_pad + seq.pad_start + q0, 512, &q_full[sq]);
                    bulk_load_1d(stat + 128, args.stat_delta + static_cast<size_t>(head) * args.S_pad + seq.pad_start + q0, 512, &q_full[sq]);
                    ok = mbar_wait(do_empty, (T & 1u) ^ 1u, abort_flag, args.status, 0x42);
                    if (!ok) break;
                    mbar_arrive_expect_tx(do_full, 2 * L::kSlab);
                    armed.arm(do_full, T & 1u);
                    for (int c = 0; c < 2; ++c)
                        tma_load_2d_chk(args.status, smem + L::kDo + c * L::kSlab, &tmap_do, do_full, head * 128 + c * 64, row_base + q0);
                }
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_st = make_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T: both K-major
            constexpr uint32_t idesc_dv = make_idesc_bf16(128, 128, 0, 1);   // dV: A = P^T (TMEM), B = dO MN-major
            constexpr uint32_t idesc_dk = make_idesc_bf16(128, 192, 0, 1);   // dK: A = dS^T (TMEM), B = Q MN-major
            // Every batch of MMAs is one asm chain (sm100_ptx.cuh): descriptors as a constant upper word and a lower
            // word that steps by immediates, commits inside the chain.  This lane's instructions cost four to six
            // clocks each beside the consumer warps and sit on the path S^T -> P^T -> dP^T -> dS^T of every tile.
            const uint64_t dk_k = desc_k_major(smem_u32(smem + L::kK)), dk_v = desc_k_major(smem_u32(smem + L::kV));
            const uint64_t dk_do = desc_k_major(smem_u32(smem + L::kDo)), dk_q0 = desc_k_major(smem_u32(smem + L::kQ));
            const uint64_t dm_do = desc_mn_major(smem_u32(smem + L::kDo), L::kSlab), dm_q0 = desc_mn_major(smem_u32(smem + L::kQ), L::kSlab);
            constexpr uint32_t kQStageLo = (3 * L::kSlab) >> 4;      // a Q stage further on, in descriptor units
            const uint32_t bars_a = smem_u32(bars);
            auto bar_a = [&](const uint64_t* b) { return bars_a + static_cast<uint32_t>(b - bars) * 8u; };
            auto issue_st = [&](uint32_t T, bool first_of_cta) -> bool {   // S^T(T) = K Q^T into X
                if (!mbar_wait(&q_full[T % L::kQStages], (T / L::kQStages) & 1u, abort_flag, args.status, 0x52)) return false;
                // X still holds dP^T of the previous tile until both groups have loaded it
                if (!first_of_cta && !mbar_wait(dp_read, (T - 1) & 1u, abort_flag, args.status, 0x57)) return false;
                tc_fence_after_sync();
                mma_ss_chain12_k128(tmem_base, desc_lo(dk_k), desc_hi(dk_k), desc_lo(dk_q0) + (T % L::kQStages) * kQStageLo, desc_hi(dk_q0),
                                    idesc_st, bar_a(st_full));
                return true;
            };
            auto issue_dp = [&](uint32_t T) -> bool {     // dP^T(T) = V dO^T over X once S^T(T) was read
                if (!mbar_wait(st_read, T & 1u, abort_flag, args.status, 0x53)) return false;
                if (!mbar_wait(do_full, T & 1u, abort_flag, args.status, 0x55)) return false;
                tc_fence_after_sync();
                mma_ss_chain8_k128(tmem_base, desc_lo(dk_v), desc_hi(dk_v), desc_lo(dk_do), desc_hi(dk_do), idesc_st, bar_a(dp_full));
                return true;
            };
            uint32_t T0 = 0;
            bool ok = true;
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_read(ring, n, true, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int t0, head, j_begin, n_iter;
                SeqTile seq;
                item_geometry(item, t0, head, j_begin, n_iter, seq);
                if (kRebuild) {
                    // the accumulator columns take the K/V tile first: the previous item's dK / dV must be drained
                    if (n > 0) ok = mbar_wait(acc_empty, (n - 1) & 1u, abort_flag, args.status, 0x58);
                    constexpr uint32_t idesc_rb = make_idesc_bf16(128, 256, 0, 1);   // A = c_kv K-major, B = W MN-major
                    for (uint32_t c = 0; c < 8u && ok; ++c) {
                        const uint32_t Tc = T0 + c, sq = Tc % L::kQStages;
                        ok = mbar_wait(&q_full[sq], (Tc / L::kQStages) & 1u, abort_flag, args.status, 0x59);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const uint32_t sa = smem_u32(smem + L::kQ + sq * 3 * L::kSlab), sb = sa + L::kSlab;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_ss(tmem_dk, desc_k_major(sa + kk * 32), desc_mn_major(sb + kk * 2048, 8192), idesc_rb,
                                   (c > 0u || kk > 0) ? 1u : 0u);
                        mma_commit(&q_empty[sq]);
                    }
                    if (ok) mma_commit(rb_full);
                    if (ok) ok = mbar_wait(kv_built, n & 1u, abort_flag, args.status, 0x5A);
                }
                if (ok) ok = mbar_wait(kv_full, n & 1u, abort_flag, args.status, 0x54);
                if (ok) ok = issue_st(T0, T0 == 0);
                if (ok) ok = issue_dp(T0);
                if (ok && n_iter == 1) mma_commit(kv_empty);
                for (int j = 0; j < n_iter && ok; ++j) {
                    const uint32_t T = T0 + j;
                    // dV += P^T(j) dO(j)   (A from Y: group 0's 64 queries, then group 1's)
                    ok = mbar_wait(p_full, T & 1u, abort_flag, args.status, 0x50);
                    // the first accumulation of an item overwrites dV and dK: the previous item's must be drained
                    if (ok && j == 0 && n > 0) ok = mbar_wait(acc_empty, (n - 1) & 1u, abort_flag, args.status, 0x56);
                    if (!ok) break;
                    tc_fence_after_sync();
                    mma_ts_chain8_mn(tmem_dv, tmem_y, desc_lo(dm_do), desc_hi(dm_do), idesc_dv, static_cast<uint32_t>(j),
                                     bar_a(do_empty), bar_a(dv_done));
                    if (j + 1 < n_iter) {
                        ok = issue_st(T + 1, false);
                        if (!ok) break;
                    }
                    // dK += dS^T(j) Q(j)
                    ok = mbar_wait(ds_full, T & 1u, abort_flag, args.status, 0x51);
                    if (!ok) break;
                    tc_fence_after_sync();
                    mma_ts_chain8_mn(tmem_dk, tmem_y, desc_lo(dm_q0) + (T % L::kQStages) * kQStageLo, desc_hi(dm_q0), idesc_dk,
                                     static_cast<uint32_t>(j), bar_a(&q_empty[T % L::kQStages]), bar_a(dk_done));
                    if (j + 1 < n_iter) {
                        ok = issue_dp(T + 1);
                        if (ok && j + 2 == n_iter) mma_commit(kv_empty);   // that was the item's last read of K and V
                    }
                }
                if (ok) mma_commit(acc_full);
                T0 += static_cast<uint32_t>(n_iter);
            }
            if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        const int g = (warp - 2) >> 2;               // consumer warpgroup: query columns [64g, 64g+64) of every tile
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;         // key row inside the tile == TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        const uint32_t tmem_x = tmem_base + lane_addr + g * 64;
        const uint32_t tmem_yg = tmem_y + lane_addr + g * 32;
        uint32_t T0 = 0;
        bool ok = true;
        for (uint32_t n = 0; ok; ++n) {
            int item = 0;
            {
                ok = mbar_wait_warp(&ring.full[n & 1u], (n >> 1) & 1u, abort_flag, args.status, 0xA1);
                if (!ok) break;
                item = ring.item[n & 1u];
                __syncwarp();
                if (lane == 0) mbar_arrive(&ring.empty[n & 1u]);
            }
            if (item < 0) break;
            int t0, head, j_begin, n_iter;
            SeqTile seq;
            item_geometry(item, t0, head, j_begin, n_iter, seq);
            const int t_idx = t0 + row;                       // key index within the sequence
            const int t_row = seq.seq_start + t_idx;          // its row in the packed tensors
            if (kRebuild) {
                // The item's K_nope / V tile is in the accumulator columns as fp32.  Group 0 rounds K_nope (columns
                // 0..127) into the two K slabs, group 1 V (128..255) into the two V slabs: row r of a slab at r * 128
                // bytes, its 16-byte chunks XORed with r & 7 -- what a 128-byte-swizzled TMA load writes.
                ok = mbar_wait_warp(rb_full, n & 1u, abort_flag, args.status, 0x66);
                if (!ok) break;
                tc_fence_after_sync();
                uint8_t* dst_row = smem + (g == 0 ? L::kK : L::kV) + row * 128;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld_x32(tmem_dk + lane_addr + g * 128 + c * 32, r);
                    tmem_ld_wait();
                    uint8_t* slab = dst_row + (c >> 1) * L::kSlab;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const int chunk = (c & 1) * 4 + v;
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(r[8 * v]), __uint_as_float(r[8 * v + 1]));
                        w.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                        w.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                        w.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                        *reinterpret_cast<uint4*>(slab + ((chunk ^ (row & 7)) << 4)) = w;
                    }
                }
                fence_async_shared();      // the MMAs and the TMA store below read the slabs through the async proxy
                tc_fence_before_sync();
                mbar_arrive(kv_built);
                if (warp == 2) {           // one lane stores the tile to the K/V workspace for the dQ kernel
                    ok = mbar_wait_warp(kv_built, n & 1u, abort_flag, args.status, 0x67);
                    if (!ok) break;
                    if (lane == 0) {
                        const int y = seq.seq_start + t0;
                        tma_store_2d(&tmap_kv, smem + L::kK, head * 256, y);
                        tma_store_2d(&tmap_kv, smem + L::kK + L::kSlab, head * 256 + 64, y);
                        tma_store_2d(&tmap_kv, smem + L::kV, head * 256 + 128, y);
                        tma_store_2d(&tmap_kv, smem + L::kV + L::kSlab, head * 256 + 192, y);
                        tma_store_commit();
                        tma_store_wait_read<0>();      // the slabs are rewritten by the next item's tile
                    }
                    __syncwarp();
                }
            }
            for (int j = 0; j < n_iter; ++j) {
                const uint32_t T = T0 + j;
                const uint32_t ph = T & 1u;
                const uint32_t sq = T % L::kQStages;
                const int q0 = (j_begin + j) * 128 + g * 64;     // first query of this group's columns
                ok = mbar_wait_warp(st_full, ph, abort_flag, args.status, 0x60);
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t sv[64];
                tmem_ld_x32(tmem_x, sv);
                tmem_ld_x32(tmem_x + 32, sv + 32);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(st_read);
                // The statistics arrived with the Q tile; waiting on its barrier here makes those bulk-copy
                // writes visible to this thread as well (the wait returns at once: S^T needed the same tile).
                ok = mbar_wait_warp(&q_full[sq], (T / L::kQStages) & 1u, abort_flag, args.status, 0x61);
                if (!ok) break;
                const float* stat = reinterpret_cast<const float*>(smem + L::kStat + sq * 1024) + g * 64;
                const bool diag = kCausal && (q0 < t0 + 128);
                float p[64];
#pragma unroll
                for (int c4 = 0; c4 < 16; ++c4) {
                    const float4 l2 = *reinterpret_cast<const float4*>(stat + c4 * 4);
                    const float l2v[4] = {l2.x, l2.y, l2.z, l2.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = c4 * 4 + e;
                        float v = fast_exp2(fmaf(__uint_as_float(sv[c]), args.scale_log2, -l2v[e]));
                        if (diag && t_idx > q0 + c) v = 0.f;
                        p[c] = v;
                    }
                }
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) pk[c] = pack_bf16x2(p[2 * c], p[2 * c + 1]);
                // Y still holds dS^T of the previous tile until dK has consumed it
                if (T > 0) {
                    ok = mbar_wait_warp(dk_done, (T - 1) & 1u, abort_flag, args.status, 0x62);
                    if (!ok) break;
                }
                tmem_st_x32(tmem_yg, pk);
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(p_full);

                ok = mbar_wait_warp(dp_full, ph, abort_flag, args.status, 0x63);
                if (!ok) break;
                tc_fence_after_sync();
                tmem_ld_x32(tmem_x, sv);
                tmem_ld_x32(tmem_x + 32, sv + 32);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(dp_read);
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    const float4 d0 = *reinterpret_cast<const float4*>(stat + 128 + c8 * 8);
                    const float4 d1 = *reinterpret_cast<const float4*>(stat + 128 + c8 * 8 + 4);
                    const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = c8 * 8 + 2 * e;
                        pk[c8 * 4 + e] = pack_bf16x2(p[c] * (__uint_as_float(sv[c]) - dl[2 * e]),
                                                     p[c + 1] * (__uint_as_float(sv[c + 1]) - dl[2 * e + 1]));
                    }
                }
                // Y holds P^T of this tile until dV has consumed it
                ok = mbar_wait_warp(dv_done, ph, abort_flag, args.status, 0x65);
                if (!ok) break;
                tmem_st_x32(tmem_yg, pk);
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(ds_full);
            }
            if (!ok) break;
            T0 += static_cast<uint32_t>(n_iter);
            ok = mbar_wait_warp(acc_full, n & 1u, abort_flag, args.status, 0x64);
            if (!ok) break;
            tc_fence_after_sync();
            const bool valid = t_idx < seq.seq_len;
            __nv_bfloat16* dkv_row = args.dkv + static_cast<size_t>(t_row) * args.h * 256 + head * 256;
            float* dkr_row = args.dkpe_acc + static_cast<size_t>(t_row) * 64;
            const bool wide = aligned32_dev(args.dkv);     // rows are h * 512 bytes: every chunk is 32-byte aligned if the base is
            // 10 chunks of 32 columns: dK nope (0..3), dK rope (4..5), dV (6..9; dV follows dK in TMEM).
            // Group 0 drains chunks 0..4, group 1 chunks 5..9.
#pragma unroll 1
            for (int c = g * 5; c < g * 5 + 5; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_x32(tmem_dk + lane_addr + c * 32, r);
                tmem_ld_wait();
                if (!valid) continue;
                if (!device_check(head < args.h && aligned16_dev(dkv_row) && aligned16_dev(dkr_row), args.status, 0xE40000u | c)) continue;
                if (c == 4 || c == 5) {
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        float4 w = make_float4(__uint_as_float(r[v * 4]) * args.scale, __uint_as_float(r[v * 4 + 1]) * args.scale,
                                               __uint_as_float(r[v * 4 + 2]) * args.scale, __uint_as_float(r[v * 4 + 3]) * args.scale);
                        if (args.dk_rope_per_head != nullptr)
                            reinterpret_cast<float4*>(args.dk_rope_per_head +
                                                      (static_cast<size_t>(head) * args.S + t_row) * 64 + (c - 4) * 32)[v] = w;
                        else
                            atomicAdd(reinterpret_cast<float4*>(dkr_row + (c - 4) * 32) + v, w);
                    }
                } else {
                    const float mul = c < 4 ? args.scale : 1.0f;
                    __nv_bfloat16* dst = dkv_row + (c < 4 ? c * 32 : 128 + (c - 6) * 32);
                    uint32_t w[16];
#pragma unroll
                    for (int v = 0; v < 16; ++v) w[v] = pack_bf16x2(__uint_as_float(r[2 * v]) * mul, __uint_as_float(r[2 * v + 1]) * mul);
                    if (wide) {          // two 32-byte stores per 32-column chunk
                        st_global_v8(dst, w);
                        st_global_v8(dst + 16, w + 8);
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            reinterpret_cast<uint4*>(dst)[v] = make_uint4(w[v * 4], w[v * 4 + 1], w[v * 4 + 2], w[v * 4 + 3]);
                    }
                }
            }
            __syncwarp();
            tc_fence_before_sync();
            mbar_arrive(acc_empty);
        }
        if (kRebuild && warp == 2 && lane == 0) tma_store_wait_all();    // the K/V tiles this lane stored are in memory
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    clock_probe_end(args.clock_probe);
}


// ================================================================================================
// dQ kernel
// ================================================================================================
struct AttnBwdDqArgs {
    int S, h;
    float scale_log2, scale;
    const float* lse;            // [S, h]
    const float* stat_delta;     // [h][S_pad]
    int S_pad;
    const __nv_bfloat16* dout;   // [S, h, 128]
    __nv_bfloat16* dq;           // [S, h, 192]
    unsigned int* status;
    WorkSchedule sched;          // items = (128-query tile, head); rank 0 = the last query tile (most keys)
    ClockProbe* clock_probe;     // may be nullptr
};

constexpr int kDqKStages = 3;

struct AttnBwdDqSmem {
    static constexpr int kSlab = 128 * 128;
    static constexpr int kQ = 0;                               // 3 slabs
    static constexpr int kK = kQ + 3 * kSlab;                  // 3 stages x 3 slabs
    static constexpr int kV = kK + kDqKStages * 3 * kSlab;     // 1 stage x 2 slabs
    static constexpr int kBar = kV + 2 * kSlab;
    static constexpr int kTotalBytes = kBar + 512;
};

// Persistent: one CTA per SM takes (query tile, head) items from the work counter.  dO of the query
// tile is the A operand of dP = dO V^T for every key tile; it is kept in TMEM as packed bf16 (64
// columns) instead of 32 KB of shared memory, which is what leaves room for a third stage of K: a K
// tile lives from its score MMA to its dQ MMA, a whole tile period later.  Between items the next
// tile's dO comes through the V stage and the MMA lane copies it to TMEM (tcgen05.cp) while the
// consumers drain the finished dQ, so the score MMAs of the next item run under the drain; the K ring
// simply keeps going across items.
template <bool kCausal>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_dq_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                         const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                         const AttnBwdDqArgs args) {
    using L = AttnBwdDqSmem;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;     // the item's last score MMA has read Q
    uint64_t* k_full = bars + 2;      // [3]
    uint64_t* k_empty = bars + 5;     // [3]
    uint64_t* v_full = bars + 8;
    uint64_t* v_empty = bars + 9;
    uint64_t* s_full = bars + 11;     // S is in TMEM
    uint64_t* s_read = bars + 12;     // both groups have loaded it
    uint64_t* dp_full = bars + 13;    // dP is in TMEM
    uint64_t* ds_full = bars + 14;    // dS (bf16) is in TMEM
    uint64_t* acc_full = bars + 15;   // the item's dQ is complete
    uint64_t* acc_empty = bars + 16;  // both groups have drained it
    ItemRing ring{bars + 17, bars + 19, reinterpret_cast<volatile int*>(bars + 21)};
    uint64_t* quiesce_bar = bars + 22;   // abort path only: the MMA lane's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 23);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1); mbar_init(q_empty, 1);
        for (int s = 0; s < kDqKStages; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
        mbar_init(v_full, 1); mbar_init(v_empty, 1);
        mbar_init(s_full, 1); mbar_init(s_read, 256); mbar_init(dp_full, 1); mbar_init(ds_full, 256);
        mbar_init(acc_full, 1); mbar_init(acc_empty, 256);
        for (int s = 0; s < 2; ++s) { mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], 9); }
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
        if ((smem_u32(smem) & 1023u) != 0u) {
            abort_flag->value = 1;
        }
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_dependency_wait();          // set-up above overlaps the previous kernel's tail; global memory from here on
    grid_launch_dependents();        // after the wait: the kernel launched behind this one starts beside it and relies on
                                     // everything before this kernel being complete (bwd_dkpe_convert_kernel)
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD1u);   // set-up found the shared memory misaligned
    clock_probe_begin(args.clock_probe);
    const uint32_t tmem_base = *tmem_slot;
    // columns: [0,128) S | [128,256) dP, then dS as bf16 (keys 0..63 in [128,160), 64..127 in [192,224)) |
    //          [256,320) dO as bf16 | [320,512) dQ
    const uint32_t tmem_dp = tmem_base + 128;
    const uint32_t tmem_do = tmem_base + 256;
    const uint32_t tmem_dq = tmem_base + 320;
    // Indices are relative to the item's sequence (see SeqTile); `seq` carries its first row, its length
    // and its start in the padded statistics arrays.
    auto item_geometry = [&](int item, int& q0, int& head, int& n_iter, SeqTile& seq) {
        int rank;
        decode_item(args.sched, item, rank, head);
        seq = seq_tile(args.sched, rank, args.S, true);        // longest rows first
        q0 = seq.tile * 128;
        n_iter = kCausal ? seq.tile + 1 : (seq.seq_len + 127) / 128;
    };

    if (abort_flag->value != 0u) {
        // misaligned shared memory: nothing was started, fall through to the common exit
    } else if (warp == 0) {
        if (elect_one()) {
            uint32_t T0 = 0;
            bool ok = true;
            ArmedBarriers armed(bars);
            auto load_k = [&](uint32_t T, int j, int head) -> bool {   // j: first row of the key tile in the packed tensors
                const uint32_t st = T % kDqKStages;
                if (!mbar_wait(&k_empty[st], ((T / kDqKStages) & 1u) ^ 1u, abort_flag, args.status, 0x70)) return false;
                mbar_arrive_expect_tx(&k_full[st], 3 * L::kSlab);
                armed.arm(&k_full[st], (T / kDqKStages) & 1u);
                uint8_t* sk = smem + L::kK + st * 3 * L::kSlab;
                tma_load_2d_chk(args.status, sk, &tmap_kv, &k_full[st], head * 256, j);
                tma_load_2d_chk(args.status, sk + L::kSlab, &tmap_kv, &k_full[st], head * 256 + 64, j);
                tma_load_2d_chk(args.status, sk + 2 * L::kSlab, &tmap_kpe, &k_full[st], 0, j);
                return true;
            };
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_publish(ring, args.sched, n, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int q0, head, n_iter;
                SeqTile seq;
                item_geometry(item, q0, head, n_iter, seq);
                const int row_base = seq.seq_start;
                ok = mbar_wait(q_empty, (n & 1u) ^ 1u, abort_flag, args.status, 0x72);
                if (!ok) break;
                mbar_arrive_expect_tx(q_full, 3 * L::kSlab);
                armed.arm(q_full, n & 1u);
                for (int c = 0; c < 3; ++c)
                    tma_load_2d_chk(args.status, smem + L::kQ + c * L::kSlab, &tmap_q, q_full, head * 192 + c * 64, row_base + q0);
                ok = load_k(T0, row_base, head);
                if (!ok) break;
                {   // The item's dO tile (the A operand of dP, kept in TMEM) goes through the single V stage ahead of the
                    // item's V tiles: 128 rows x 128 elements are exactly its two slabs.  The MMA lane copies it to TMEM
                    // (tcgen05.cp).  One more entry per item: the stage's barriers are counted on T + n.
                    const uint32_t ph = (T0 + n) & 1u;
                    ok = mbar_wait(v_empty, ph ^ 1u, abort_flag, args.status, 0x73);
                    if (!ok) break;
                    mbar_arrive_expect_tx(v_full, 2 * L::kSlab);
                    armed.arm(v_full, ph);
                    tma_load_2d_chk(args.status, smem + L::kV, &tmap_do, v_full, head * 128, row_base + q0);
                    tma_load_2d_chk(args.status, smem + L::kV + L::kSlab, &tmap_do, v_full, head * 128 + 64, row_base + q0);
                }
                for (int j = 0; j < n_iter && ok; ++j) {
                    const uint32_t T = T0 + j;
                    if (j + 1 < n_iter) ok = load_k(T + 1, row_base + (j + 1) * 128, head);
                    if (!ok) break;
                    const uint32_t phv = (T + n + 1u) & 1u;
                    ok = mbar_wait(v_empty, phv ^ 1u, abort_flag, args.status, 0x71);
                    if (!ok) break;
                    mbar_arrive_expect_tx(v_full, 2 * L::kSlab);
                    armed.arm(v_full, phv);
                    tma_load_2d_chk(args.status, smem + L::kV, &tmap_kv, v_full, head * 256 + 128, row_base + j * 128);
                    tma_load_2d_chk(args.status, smem + L::kV + L::kSlab, &tmap_kv, v_full, head * 256 + 192, row_base + j * 128);
                }
                T0 += static_cast<uint32_t>(n_iter);
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);    // S: both K-major; dP: A from TMEM
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 192, 0, 1);   // dQ: A = dS (TMEM), B = K MN-major
            // (one asm chain per batch of MMAs, as in the dK/dV kernel)
            const uint64_t dk_q = desc_k_major(smem_u32(smem + L::kQ)), dk_v = desc_k_major(smem_u32(smem + L::kV));
            const uint64_t dk_k0 = desc_k_major(smem_u32(smem + L::kK)), dm_k0 = desc_mn_major(smem_u32(smem + L::kK), L::kSlab);
            constexpr uint32_t kKStageLo = (3 * L::kSlab) >> 4;      // a K stage further on, in descriptor units
            const uint32_t bars_a = smem_u32(bars);
            auto bar_a = [&](const uint64_t* b) { return bars_a + static_cast<uint32_t>(b - bars) * 8u; };
            auto issue_s = [&](uint32_t T) -> bool {      // S(T) = Q K^T
                if (!mbar_wait(&k_full[T % kDqKStages], (T / kDqKStages) & 1u, abort_flag, args.status, 0x82)) return false;
                if (T > 0 && !mbar_wait(s_read, (T - 1) & 1u, abort_flag, args.status, 0x83)) return false;
                tc_fence_after_sync();
                mma_ss_chain12_k128(tmem_base, desc_lo(dk_q), desc_hi(dk_q), desc_lo(dk_k0) + (T % kDqKStages) * kKStageLo, desc_hi(dk_k0),
                                    idesc_s, bar_a(s_full));
                return true;
            };
            auto issue_dp = [&](uint32_t T, uint32_t n) -> bool {     // dP(T) = dO V^T; overwrites dS(T-1), whose reader was issued earlier
                if (!mbar_wait(v_full, (T + n + 1u) & 1u, abort_flag, args.status, 0x84)) return false;
                tc_fence_after_sync();
                mma_ts_chain8_k128(tmem_dp, tmem_do, desc_lo(dk_v), desc_hi(dk_v), idesc_s, bar_a(v_empty), bar_a(dp_full));
                return true;
            };
            uint32_t T0 = 0;
            bool ok = true;
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_read(ring, n, true, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int q0, head, n_iter;
                SeqTile seq;
                item_geometry(item, q0, head, n_iter, seq);
                ok = mbar_wait(q_full, n & 1u, abort_flag, args.status, 0x81);
                if (ok) ok = issue_s(T0);
                if (ok && n_iter == 1) mma_commit(q_empty);
                if (ok) {     // the item's dO tile: from the V stage to TMEM (every dP MMA of the previous item has completed:
                              // its last dS, which this lane has consumed, was computed from the last of them)
                    ok = mbar_wait(v_full, (T0 + n) & 1u, abort_flag, args.status, 0x85);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t sv = smem_u32(smem + L::kV);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            tmem_cp_128x256b(tmem_do + kk * 8, desc_k_major(sv + (kk >> 2) * L::kSlab + (kk & 3) * 32));
                        mma_commit(v_empty);
                    }
                }
                if (ok) ok = issue_dp(T0, n);
                for (int j = 0; j < n_iter && ok; ++j) {
                    const uint32_t T = T0 + j;
                    if (j + 1 < n_iter) {
                        ok = issue_s(T + 1);
                        if (ok && j + 2 == n_iter) mma_commit(q_empty);   // that was the item's last read of Q
                    }
                    if (!ok) break;
                    ok = mbar_wait(ds_full, T & 1u, abort_flag, args.status, 0x80);
                    // the first accumulation of an item overwrites dQ: the previous item's must be drained
                    if (ok && j == 0 && n > 0) ok = mbar_wait(acc_empty, (n - 1) & 1u, abort_flag, args.status, 0x86);
                    if (!ok) break;
                    tc_fence_after_sync();
                    mma_ts_chain8_mn_split(tmem_dq, tmem_dp, desc_lo(dm_k0) + (T % kDqKStages) * kKStageLo, desc_hi(dm_k0), idesc_dq,
                                           static_cast<uint32_t>(j), bar_a(&k_empty[T % kDqKStages]));
                    if (j + 1 < n_iter) ok = issue_dp(T + 1, n);
                }
                if (ok) mma_commit(acc_full);
                T0 += static_cast<uint32_t>(n_iter);
            }
            if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        const int g = (warp - 2) >> 2;               // consumer group: key columns [64g, 64g+64) of the tile
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        auto read_item = [&](uint32_t n, bool& ok) -> int {
            ok = mbar_wait_warp(&ring.full[n & 1u], (n >> 1) & 1u, abort_flag, args.status, 0xA1);
            if (!ok) return -1;
            const int it = ring.item[n & 1u];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ring.empty[n & 1u]);
            return it;
        };
        // dQ of a finished item: six 32-column chunks, three per group
        // (s_idx: the row in the packed tensors; valid: it lies inside its sequence)
        auto drain = [&](uint32_t n_done, int s_idx, bool valid, int head) -> bool {
            if (!mbar_wait_warp(acc_full, n_done & 1u, abort_flag, args.status, 0x92)) return false;
            tc_fence_after_sync();
            __nv_bfloat16* dst = args.dq + (static_cast<size_t>(s_idx) * args.h + head) * 192;
            const bool wide = aligned32_dev(args.dq);      // rows are 384 bytes: every chunk is 32-byte aligned if the base is
#pragma unroll 1
            for (int c = g * 3; c < g * 3 + 3; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_x32(tmem_dq + lane_addr + c * 32, r);
                tmem_ld_wait();
                if (!valid) continue;
                if (!device_check(head < args.h && aligned16_dev(dst), args.status, 0xE50000u | c)) continue;
                uint32_t w[16];
#pragma unroll
                for (int v = 0; v < 16; ++v) w[v] = pack_bf16x2(__uint_as_float(r[2 * v]) * args.scale, __uint_as_float(r[2 * v + 1]) * args.scale);
                if (wide) {          // two 32-byte stores per 32-column chunk
                    st_global_v8(dst + c * 32, w);
                    st_global_v8(dst + c * 32 + 16, w + 8);
                } else {
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        reinterpret_cast<uint4*>(dst + c * 32)[v] = make_uint4(w[v * 4], w[v * 4 + 1], w[v * 4 + 2], w[v * 4 + 3]);
                }
            }
            __syncwarp();
            tc_fence_before_sync();
            mbar_arrive(acc_empty);
            return true;
        };
        uint32_t T0 = 0;
        bool ok = true;
        int item = read_item(0, ok);
        int prev_s_idx = 0, prev_head = 0;
        bool prev_valid = false;
        for (uint32_t n = 0; ok && item >= 0; ++n) {
            int q0, head, n_iter;
            SeqTile seq;
            item_geometry(item, q0, head, n_iter, seq);
            const int S_seq = seq.seq_len;
            const int s_idx = q0 + row;                       // query index within the sequence
            const int s_row = seq.seq_start + s_idx;          // its row in the packed tensors
            const bool valid = s_idx < S_seq;
            // Rows past the end of the sequence get LSE = +inf so that their P is exactly zero.
            const float l2 = valid ? args.lse[static_cast<size_t>(s_row) * args.h + head] * 1.4426950408889634f : INFINITY;
            const float delta = valid ? args.stat_delta[static_cast<size_t>(head) * args.S_pad + seq.pad_start + s_idx] : 0.f;
            if (n > 0) ok = drain(n - 1, prev_s_idx, prev_valid, prev_head);
            for (int j = 0; j < n_iter && ok; ++j) {
                const uint32_t T = T0 + j;
                ok = mbar_wait_warp(s_full, T & 1u, abort_flag, args.status, 0x90);
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t sv[64];
                tmem_ld_x32(tmem_base + lane_addr + g * 64, sv);
                tmem_ld_x32(tmem_base + lane_addr + g * 64 + 32, sv + 32);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(s_read);
                const int tk0 = j * 128 + g * 64;
                const bool edge = (kCausal && tk0 + 63 > q0) || (tk0 + 64 > S_seq);
                float p[64];
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    float v = fast_exp2(fmaf(__uint_as_float(sv[c]), args.scale_log2, -l2));
                    if (edge) {
                        const int t = tk0 + c;
                        if ((kCausal && t > s_idx) || t >= S_seq) v = 0.f;
                    }
                    p[c] = v;
                }
                ok = mbar_wait_warp(dp_full, T & 1u, abort_flag, args.status, 0x91);
                if (!ok) break;
                tc_fence_after_sync();
                tmem_ld_x32(tmem_dp + lane_addr + g * 64, sv);
                tmem_ld_x32(tmem_dp + lane_addr + g * 64 + 32, sv + 32);
                tmem_ld_wait();
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    pk[c] = pack_bf16x2(p[2 * c] * (__uint_as_float(sv[2 * c]) - delta),
                                        p[2 * c + 1] * (__uint_as_float(sv[2 * c + 1]) - delta));
                tmem_st_x32(tmem_dp + lane_addr + g * 64, pk);   // dS over the first 32 columns of this group's own half
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(ds_full);
            }
            if (!ok) break;
            T0 += static_cast<uint32_t>(n_iter);
            prev_s_idx = s_row;
            prev_valid = valid;
            prev_head = head;
            item = read_item(n + 1, ok);
            if (ok && item < 0) ok = drain(n, prev_s_idx, prev_valid, prev_head);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    clock_probe_end(args.clock_probe);
}

}  // namespace laga
