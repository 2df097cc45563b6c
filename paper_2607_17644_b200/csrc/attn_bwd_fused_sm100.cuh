// Backward of Algorithm 1 step 5 (Section 5.2) in ONE pass over the score tiles, on CTA pairs.
//
// The two-kernel backward (attn_bwd_sm100.cuh) computes S and dP twice: once with keys stationary for
// dK / dV, once with queries stationary for dQ.  Five 128x128 products per tile pair are needed
// (S^T, dP^T, dV, dK, dQ) but seven are executed.  Here a cluster of two CTAs shares one (128-key tile,
// head) item and executes exactly the five, split so that each SM's tensor pipe gets the same load:
//
//   "score" CTA (cluster rank 0)                     "gradient" CTA (cluster rank 1)
//     S^T  = K Q^T            (768 clocks)              dQ^T = [K_nope | k_pe]^T dS^T   (1024: 768 useful;
//     dP^T = V dO^T           (512)                              the 64 rope rows run as a 128-row MMA)
//     P^T  = exp2(scale S^T - LSE), dS^T = P^T (dP^T - delta)   dK  += dS^T Q             (768)
//     dV  += P^T dO           (512)
//
// dS^T (bf16, 128 keys x 128 queries) crosses from the score CTA to the gradient CTA through distributed
// shared memory: every consumer thread of the score CTA stores its key row (2 x 128 bytes, in the
// 128-byte-swizzled layout the MMAs read) into the peer's buffer and arrives on the peer's barrier; the
// gradient CTA's MMA lane tells the score CTA that a buffer is free again with a tcgen05.commit that arrives
// on the peer's barrier.  The same buffer serves as the K-major A operand of dK and the MN-major B operand
// of dQ^T, so nothing is transposed anywhere.
//
// dQ: a (key tile, head) item only holds one key tile's contribution to each query row, so dQ^T tiles are
// added into an fp32 accumulator in global memory, dq_acc[S][heads of this launch][192], with red.add
// (TMEM lanes are the 192 channels: one warp instruction adds 32 consecutive floats = one 128-byte line),
// and a small kernel afterwards scales, rounds to bf16 and clears the accumulator.  The accumulator is why a
// launch covers a window of heads: the host sizes the window so that it stays L2 resident.
// Floating-point addition order in dq_acc depends on timing, so dQ is not bit-reproducible run to run;
// the deterministic flag of the C interface selects the two-kernel path instead.
//
// Work distribution is static: items of the launch are ordered longest first (key tile 0 of every head, then
// key tile 1, ...) and pair p takes items p, p + pairs, p + 2 pairs, ... -- both CTAs of a pair derive the
// same sequence on their own.  Tiles of consecutive items form one stream per CTA (a running tile count T
// gives every ring its slot and phase), so the score MMAs of an item's first tile are issued while the
// previous item's last tile is still in the softmax.
#pragma once
#include "attn_bwd_sm100.cuh"
#include "sm100_ptx.cuh"
#include "work_sched.cuh"

namespace laga {

struct AttnBwdFusedArgs {
    int S, h, S_pad;
    int head_begin, head_count;   // the heads this launch covers
    float scale_log2, scale;
    const float* stat_l2;         // [h][S_pad]  LSE * log2(e), +inf past S
    const float* stat_delta;      // [h][S_pad]
    const __nv_bfloat16* kv;      // [S, h*256]  (the score CTA copies its V rows into TMEM itself)
    __nv_bfloat16* dkv;           // [S, h*256]: per head dK_nope (128) then dV (128)
    float* dkpe_acc;              // [S][64] fp32, zero before the first launch of a backward pass
    float* dq_acc;                // [S][head_count][192] fp32, zero when the kernel starts; unscaled sums
    unsigned int* status;
    ClockProbe* clock_probe;      // may be nullptr
};

struct AttnBwdFusedSmem {
    static constexpr int kSlab = 128 * 128;                    // 128 rows x 128 B
    static constexpr int kK = 0;                               // both roles: K_nope (2 slabs) + rope band (1)
    // score CTA
    static constexpr int kQs = kK + 3 * kSlab;                 // 2 stages x 3 slabs
    static constexpr int kDo = kQs + 2 * 3 * kSlab;            // 2 stages x 2 slabs
    // gradient CTA
    static constexpr int kDs = kK + 3 * kSlab;                 // 2 buffers x 2 slabs (written by the peer)
    static constexpr int kQg = kDs + 2 * 2 * kSlab;            // 2 stages x 3 slabs
    static constexpr int kStat = kK + 13 * kSlab;              // score CTA: 4 stages x (128 l2 + 128 delta floats)
    static constexpr int kBar = kStat + 4 * 1024;
    static constexpr int kTotalBytes = kBar + 512;
};
static_assert(AttnBwdFusedSmem::kDo + 2 * 2 * AttnBwdFusedSmem::kSlab == AttnBwdFusedSmem::kStat, "score CTA layout");
static_assert(AttnBwdFusedSmem::kQg + 2 * 3 * AttnBwdFusedSmem::kSlab == AttnBwdFusedSmem::kStat, "gradient CTA layout");
static_assert(AttnBwdFusedSmem::kTotalBytes <= 232448, "fused backward exceeds the 227 KB of shared memory per CTA");

// One position in a CTA's tile stream.
struct FusedTile {
    int n;        // item number of this pair (0, 1, ...)
    int j;        // tile within the item
    int n_iter;   // tiles of the item
    int head, t0, j_begin;
    bool valid;
};

template <bool kCausal>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kBwdThreads, 1)
attn_bwd_fused_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                            const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                            const AttnBwdFusedArgs args) {
    using L = AttnBwdFusedSmem;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    // Barriers of both roles live at the same offsets in both CTAs (a commit that signals the peer names an offset).
    uint64_t* k_full = bars + 0;        // per item
    uint64_t* k_empty = bars + 1;
    uint64_t* q_full = bars + 2;        // [2]
    uint64_t* q_empty = bars + 4;       // [2]
    uint64_t* do_full = bars + 6;       // [2]  score CTA
    uint64_t* do_empty = bars + 8;      // [2]
    uint64_t* stat_full = bars + 10;    // [4]  score CTA: LSE / delta of a query tile
    uint64_t* stat_empty = bars + 14;   // [4]  count 8: one lane per consumer warp, after dS^T of the tile
    uint64_t* st_full = bars + 18;      // [2]  per X buffer: S^T is in it
    uint64_t* st_read = bars + 20;      // [2]  count 256: the consumers loaded it, dP^T may overwrite it
    uint64_t* dp_full = bars + 22;      // [2]  dP^T is in the buffer
    uint64_t* dp_read = bars + 24;      // [2]  count 256: loaded, the buffer may take the S^T after next
    uint64_t* p_full = bars + 26;       // count 256: P^T (bf16) is in Y
    uint64_t* dv_done = bars + 27;      // dV += P^T dO has read Y
    uint64_t* v_ready = bars + 28;      // count 256: the item's V is in TMEM
    uint64_t* acc_full = bars + 29;     // the item's dV (score CTA) / dK (gradient CTA) is complete
    uint64_t* acc_empty = bars + 30;    // count 256: drained
    uint64_t* ds_free = bars + 31;      // [2]  in the SCORE CTA, signalled by the gradient CTA's commit: buffer reusable
    uint64_t* ds_full = bars + 33;      // [2]  in the GRADIENT CTA, count 256, signalled by the score CTA's consumers
    uint64_t* dq_full = bars + 35;      // gradient CTA: dQ^T of the tile is in TMEM
    uint64_t* dq_read = bars + 36;      // count 256: loaded, the next dQ^T may overwrite it
    uint64_t* quiesce_bar = bars + 37;  // abort path only
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 38);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t role = cluster_cta_rank();          // 0 = score CTA, 1 = gradient CTA
    const int n_q128 = (args.S + 127) / 128;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int total_items = n_q128 * args.head_count;

    if (threadIdx.x == 0) {
        mbar_init(k_full, 1); mbar_init(k_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1);
            mbar_init(&do_full[s], 1); mbar_init(&do_empty[s], 1);
            mbar_init(&st_full[s], 1); mbar_init(&st_read[s], 256);
            mbar_init(&dp_full[s], 1); mbar_init(&dp_read[s], 256);
            mbar_init(&ds_free[s], 1); mbar_init(&ds_full[s], 256);
        }
        for (int s = 0; s < 4; ++s) { mbar_init(&stat_full[s], 1); mbar_init(&stat_empty[s], 8); }
        mbar_init(p_full, 256); mbar_init(dv_done, 1); mbar_init(v_ready, 256);
        mbar_init(acc_full, 1); mbar_init(acc_empty, 256);
        mbar_init(dq_full, 1); mbar_init(dq_read, 256);
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
    cluster_sync();                      // the peer's barriers are initialised before anything arrives on them
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();              // global memory from here on
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD2u);   // set-up found the shared memory misaligned
    clock_probe_begin(args.clock_probe);
    const uint32_t tmem_base = *tmem_slot;

    auto tile_at = [&](int n) -> FusedTile {
        FusedTile t;
        t.n = n; t.j = 0;
        const long long item = static_cast<long long>(pair) + static_cast<long long>(n) * n_pairs;
        t.valid = item < total_items;
        const int it = t.valid ? static_cast<int>(item) : 0;
        const int k_tile = it / args.head_count;
        t.head = args.head_begin + (it - k_tile * args.head_count);
        t.t0 = k_tile * 128;
        t.j_begin = kCausal ? k_tile : 0;
        t.n_iter = n_q128 - t.j_begin;           // >= 1
        return t;
    };
    auto advance = [&](FusedTile& t) {
        if (++t.j == t.n_iter) t = tile_at(t.n + 1);
    };

    if (abort_flag->value != 0u) {
        // misaligned shared memory: nothing was started, fall through to the common exit
    } else if (role == 0) {
        // ========================================= score CTA =========================================
        // TMEM columns: [0,128) dV | [128,256) X0 | [256,384) X1 | [384,448) Y (P^T, bf16) | [448,512) V (bf16)
        const uint32_t tmem_dv = tmem_base;
        const uint32_t tmem_y = tmem_base + 384;
        const uint32_t tmem_v = tmem_base + 448;
        if (warp == 0) {
            if (elect_one()) {
                ArmedBarriers armed(bars);
                uint32_t T = 0;
                bool ok = true;
                for (FusedTile it = tile_at(0); it.valid && ok; it = tile_at(it.n + 1)) {
                    ok = mbar_wait(k_empty, (it.n & 1u) ^ 1u, abort_flag, args.status, 0x1A0);
                    if (!ok) break;
                    mbar_arrive_expect_tx(k_full, 3 * L::kSlab);
                    armed.arm(k_full, it.n & 1u);
                    tma_load_2d_chk(args.status, smem + L::kK, &tmap_kv, k_full, it.head * 256, it.t0);
                    tma_load_2d_chk(args.status, smem + L::kK + L::kSlab, &tmap_kv, k_full, it.head * 256 + 64, it.t0);
                    tma_load_2d_chk(args.status, smem + L::kK + 2 * L::kSlab, &tmap_kpe, k_full, 0, it.t0);
                    for (int j = 0; j < it.n_iter; ++j, ++T) {
                        const uint32_t s2 = T & 1u, ph2 = (T >> 1) & 1u, s4 = T & 3u, ph4 = (T >> 2) & 1u;
                        const int q0 = (it.j_begin + j) * 128;
                        ok = mbar_wait(&q_empty[s2], ph2 ^ 1u, abort_flag, args.status, 0x1A1);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&q_full[s2], 3 * L::kSlab);
                        armed.arm(&q_full[s2], ph2);
                        for (int c = 0; c < 3; ++c)
                            tma_load_2d_chk(args.status, smem + L::kQs + (s2 * 3 + c) * L::kSlab, &tmap_q, &q_full[s2],
                                            it.head * 192 + c * 64, q0);
                        ok = mbar_wait(&stat_empty[s4], ph4 ^ 1u, abort_flag, args.status, 0x1A2);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&stat_full[s4], 1024);
                        armed.arm(&stat_full[s4], ph4);
                        float* stat = reinterpret_cast<float*>(smem + L::kStat + s4 * 1024);
                        bulk_load_1d(stat, args.stat_l2 + static_cast<size_t>(it.head) * args.S_pad + q0, 512, &stat_full[s4]);
                        bulk_load_1d(stat + 128, args.stat_delta + static_cast<size_t>(it.head) * args.S_pad + q0, 512, &stat_full[s4]);
                        ok = mbar_wait(&do_empty[s2], ph2 ^ 1u, abort_flag, args.status, 0x1A3);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&do_full[s2], 2 * L::kSlab);
                        armed.arm(&do_full[s2], ph2);
                        for (int c = 0; c < 2; ++c)
                            tma_load_2d_chk(args.status, smem + L::kDo + (s2 * 2 + c) * L::kSlab, &tmap_do, &do_full[s2],
                                            it.head * 128 + c * 64, q0);
                    }
                }
                if (abort_flag->value != 0u) armed.quiesce();
            }
        } else if (warp == 1) {
            if (elect_one()) {
                constexpr uint32_t idesc_st = make_idesc_bf16(128, 128, 0, 0);   // S^T (SS) and dP^T (A = V in TMEM)
                constexpr uint32_t idesc_dv = make_idesc_bf16(128, 128, 0, 1);   // dV: A = P^T (TMEM), B = dO MN-major
                const uint32_t sk = smem_u32(smem + L::kK);
                auto issue_st = [&](const FusedTile& it, uint32_t T) -> bool {   // S^T(T) = K Q^T into X[T & 1]
                    const uint32_t b = T & 1u, ph = (T >> 1) & 1u;
                    if (it.j == 0 && !mbar_wait(k_full, it.n & 1u, abort_flag, args.status, 0x1B0)) return false;
                    if (!mbar_wait(&q_full[b], ph, abort_flag, args.status, 0x1B1)) return false;
                    // the buffer holds dP^T of tile T-2 until both groups have loaded it
                    if (T >= 2u && !mbar_wait(&dp_read[b], ph ^ 1u, abort_flag, args.status, 0x1B2)) return false;
                    tc_fence_after_sync();
                    const uint32_t sq = smem_u32(smem + L::kQs + b * 3 * L::kSlab);
                    const uint32_t tmem_x = tmem_base + 128 + b * 128;
#pragma unroll
                    for (int kk = 0; kk < 12; ++kk) {
                        const uint32_t off = (kk >> 2) * L::kSlab + (kk & 3) * 32;
                        mma_ss(tmem_x, desc_k_major(sk + off), desc_k_major(sq + off), idesc_st, kk > 0 ? 1u : 0u);
                    }
                    mma_commit(&st_full[b]);
                    mma_commit(&q_empty[b]);
                    if (it.j + 1 == it.n_iter) mma_commit(k_empty);   // the item's last read of K
                    return true;
                };
                auto issue_dp = [&](const FusedTile& it, uint32_t T) -> bool {   // dP^T(T) = V dO^T over X[T & 1]
                    const uint32_t b = T & 1u, ph = (T >> 1) & 1u;
                    if (it.j == 0 && !mbar_wait(v_ready, it.n & 1u, abort_flag, args.status, 0x1B3)) return false;
                    if (!mbar_wait(&st_read[b], ph, abort_flag, args.status, 0x1B4)) return false;
                    if (!mbar_wait(&do_full[b], ph, abort_flag, args.status, 0x1B5)) return false;
                    tc_fence_after_sync();
                    const uint32_t sdo = smem_u32(smem + L::kDo + b * 2 * L::kSlab);
                    const uint32_t tmem_x = tmem_base + 128 + b * 128;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_ts(tmem_x, tmem_v + kk * 8, desc_k_major(sdo + (kk >> 2) * L::kSlab + (kk & 3) * 32), idesc_st,
                               kk > 0 ? 1u : 0u);
                    mma_commit(&dp_full[b]);
                    return true;
                };
                auto issue_dv = [&](const FusedTile& it, uint32_t T) -> bool {   // dV += P^T(T) dO(T)
                    const uint32_t b = T & 1u;
                    if (!mbar_wait(p_full, T & 1u, abort_flag, args.status, 0x1B6)) return false;
                    // the first accumulation of an item overwrites dV: the previous item's must be drained
                    if (it.j == 0 && it.n > 0 && !mbar_wait(acc_empty, (it.n - 1) & 1u, abort_flag, args.status, 0x1B7)) return false;
                    tc_fence_after_sync();
                    const uint32_t sdo = smem_u32(smem + L::kDo + b * 2 * L::kSlab);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_ts(tmem_dv, tmem_y + kk * 8, desc_mn_major(sdo + kk * 2048, L::kSlab), idesc_dv,
                               (it.j > 0 || kk > 0) ? 1u : 0u);
                    mma_commit(&do_empty[b]);
                    mma_commit(dv_done);
                    if (it.j + 1 == it.n_iter) mma_commit(acc_full);
                    return true;
                };
                FusedTile cur = tile_at(0);
                uint32_t T = 0;
                bool ok = !cur.valid || issue_st(cur, 0);
                while (ok && cur.valid) {
                    FusedTile nxt = cur;
                    advance(nxt);
                    ok = issue_dp(cur, T);
                    if (ok && nxt.valid) ok = issue_st(nxt, T + 1);
                    if (ok) ok = issue_dv(cur, T);
                    cur = nxt;
                    ++T;
                }
                if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
            }
        } else {
            const int g = (warp - 2) >> 2;               // consumer warpgroup: query columns [64g, 64g+64) of every tile
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;         // key row inside the tile == TMEM lane
            const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
            const uint32_t tmem_yg = tmem_y + lane_addr + g * 32;
            // this thread's row of the peer's dS^T buffers: slab g (64 queries), 128 bytes, chunk c at c ^ (row & 7)
            const uint32_t ds_peer = cluster_map(smem + L::kDs, 1u) + g * L::kSlab + row * 128;
            const uint32_t ds_full_peer = cluster_map(ds_full, 1u);
            auto drain = [&](int n_done, int t_idx, int head) -> bool {     // dV of a finished item: 2 chunks per group
                if (!mbar_wait_warp(acc_full, n_done & 1u, abort_flag, args.status, 0x1C6)) return false;
                tc_fence_after_sync();
                const bool valid = t_idx < args.S;
                __nv_bfloat16* dst = args.dkv + static_cast<size_t>(t_idx) * args.h * 256 + head * 256 + 128;
#pragma unroll 1
                for (int c = g * 2; c < g * 2 + 2; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld_x32(tmem_dv + lane_addr + c * 32, r);
                    tmem_ld_wait();
                    if (!valid) continue;
                    if (!device_check(head < args.h && aligned16_dev(dst), args.status, 0xE60000u | c)) continue;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
                        w.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
                        w.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
                        w.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
                        reinterpret_cast<uint4*>(dst + c * 32)[v] = w;
                    }
                }
                __syncwarp();
                tc_fence_before_sync();
                mbar_arrive(acc_empty);
                return true;
            };
            uint32_t T = 0;
            bool ok = true;
            int prev_t_idx = 0, prev_head = 0;
            FusedTile it = tile_at(0);
            while (ok && it.valid) {
                const int t_idx = it.t0 + row;
                const bool row_live = t_idx < args.S;
                {   // this thread's V row, channels [64g, 64g+64), as 32 packed words into TMEM (the previous item's
                    // last dP^T has completed: this group waited for it before computing its last dS^T)
                    uint32_t w[32];
                    if (row_live) {
                        const uint4* src = reinterpret_cast<const uint4*>(args.kv + static_cast<size_t>(t_idx) * args.h * 256 +
                                                                          it.head * 256 + 128 + g * 64);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const uint4 x = src[v];
                            w[v * 4] = x.x; w[v * 4 + 1] = x.y; w[v * 4 + 2] = x.z; w[v * 4 + 3] = x.w;
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < 32; ++v) w[v] = 0u;
                    }
                    __syncwarp();
                    tmem_st_x32(tmem_v + lane_addr + g * 32, w);
                    tmem_st_wait();
                    tc_fence_before_sync();
                    mbar_arrive(v_ready);
                }
                if (it.n > 0) ok = drain(it.n - 1, prev_t_idx, prev_head);
                for (int j = 0; j < it.n_iter && ok; ++j, ++T) {
                    const uint32_t b = T & 1u, ph = (T >> 1) & 1u, s4 = T & 3u;
                    const uint32_t tmem_x = tmem_base + 128 + b * 128 + lane_addr + g * 64;
                    const int q0 = (it.j_begin + j) * 128 + g * 64;     // first query of this group's columns
                    ok = mbar_wait_warp(&st_full[b], ph, abort_flag, args.status, 0x1C0);
                    if (!ok) break;
                    tc_fence_after_sync();
                    uint32_t sv[64];
                    tmem_ld_x32(tmem_x, sv);
                    tmem_ld_x32(tmem_x + 32, sv + 32);
                    tmem_ld_wait();
                    tc_fence_before_sync();
                    mbar_arrive(&st_read[b]);
                    ok = mbar_wait_warp(&stat_full[s4], (T >> 2) & 1u, abort_flag, args.status, 0x1C1);
                    if (!ok) break;
                    const float* stat = reinterpret_cast<const float*>(smem + L::kStat + s4 * 1024) + g * 64;
                    const bool diag = kCausal && (q0 < it.t0 + 128);
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
                            // key rows past the end of the sequence must not reach dQ (their K rows are zero, not -inf)
                            p[c] = row_live ? v : 0.f;
                        }
                    }
                    uint32_t pk[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) pk[c] = pack_bf16x2(p[2 * c], p[2 * c + 1]);
                    // Y still holds P^T of the previous tile until its dV has consumed it
                    if (T > 0) {
                        ok = mbar_wait_warp(dv_done, (T - 1) & 1u, abort_flag, args.status, 0x1C2);
                        if (!ok) break;
                    }
                    tmem_st_x32(tmem_yg, pk);
                    tmem_st_wait();
                    tc_fence_before_sync();
                    mbar_arrive(p_full);
                    ok = mbar_wait_warp(&dp_full[b], ph, abort_flag, args.status, 0x1C3);
                    if (!ok) break;
                    tc_fence_after_sync();
                    tmem_ld_x32(tmem_x, sv);
                    tmem_ld_x32(tmem_x + 32, sv + 32);
                    tmem_ld_wait();
                    tc_fence_before_sync();
                    mbar_arrive(&dp_read[b]);
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
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&stat_empty[s4]);
                    // the peer's buffer is free once its dK MMAs of tile T-2 have completed
                    ok = mbar_wait_warp(&ds_free[b], ph ^ 1u, abort_flag, args.status, 0x1C4);
                    if (!ok) break;
                    const uint32_t dst = ds_peer + b * 2 * L::kSlab;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        st_shared_cluster_v4(dst + ((c ^ (row & 7)) << 4), make_uint4(pk[c * 4], pk[c * 4 + 1], pk[c * 4 + 2], pk[c * 4 + 3]));
                    fence_proxy_async_all();
                    mbar_arrive_cluster(ds_full_peer + b * 8);
                }
                if (!ok) break;
                prev_t_idx = t_idx;
                prev_head = it.head;
                const int n_done = it.n;
                it = tile_at(it.n + 1);
                if (!it.valid) ok = drain(n_done, prev_t_idx, prev_head);
            }
        }
    } else {
        // ======================================== gradient CTA ========================================
        // TMEM columns: [0,192) dK | [192,320) dQ^T nope channels | [320,448) dQ^T rope channels (lanes 0..63)
        const uint32_t tmem_dk = tmem_base;
        const uint32_t tmem_dqn = tmem_base + 192;
        const uint32_t tmem_dqr = tmem_base + 320;
        if (warp == 0) {
            if (elect_one()) {
                ArmedBarriers armed(bars);
                uint32_t T = 0;
                bool ok = true;
                for (FusedTile it = tile_at(0); it.valid && ok; it = tile_at(it.n + 1)) {
                    ok = mbar_wait(k_empty, (it.n & 1u) ^ 1u, abort_flag, args.status, 0x1D0);
                    if (!ok) break;
                    mbar_arrive_expect_tx(k_full, 3 * L::kSlab);
                    armed.arm(k_full, it.n & 1u);
                    tma_load_2d_chk(args.status, smem + L::kK, &tmap_kv, k_full, it.head * 256, it.t0);
                    tma_load_2d_chk(args.status, smem + L::kK + L::kSlab, &tmap_kv, k_full, it.head * 256 + 64, it.t0);
                    tma_load_2d_chk(args.status, smem + L::kK + 2 * L::kSlab, &tmap_kpe, k_full, 0, it.t0);
                    for (int j = 0; j < it.n_iter; ++j, ++T) {
                        const uint32_t s2 = T & 1u, ph2 = (T >> 1) & 1u;
                        const int q0 = (it.j_begin + j) * 128;
                        ok = mbar_wait(&q_empty[s2], ph2 ^ 1u, abort_flag, args.status, 0x1D1);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&q_full[s2], 3 * L::kSlab);
                        armed.arm(&q_full[s2], ph2);
                        for (int c = 0; c < 3; ++c)
                            tma_load_2d_chk(args.status, smem + L::kQg + (s2 * 3 + c) * L::kSlab, &tmap_q, &q_full[s2],
                                            it.head * 192 + c * 64, q0);
                    }
                }
                if (abort_flag->value != 0u) armed.quiesce();
            }
        } else if (warp == 1) {
            if (elect_one()) {
                constexpr uint32_t idesc_dq = make_idesc_bf16(128, 128, 1, 1);   // dQ^T: A = K (MN-major), B = dS^T (MN-major)
                constexpr uint32_t idesc_dk = make_idesc_bf16(128, 192, 0, 1);   // dK: A = dS^T (K-major), B = Q (MN-major)
                const uint32_t sk = smem_u32(smem + L::kK);
                uint32_t T = 0;
                bool ok = true;
                for (FusedTile it = tile_at(0); it.valid && ok; it = tile_at(it.n + 1)) {
                    ok = mbar_wait(k_full, it.n & 1u, abort_flag, args.status, 0x1E0);
                    for (int j = 0; j < it.n_iter && ok; ++j, ++T) {
                        const uint32_t b = T & 1u, ph = (T >> 1) & 1u;
                        const uint32_t sds = smem_u32(smem + L::kDs + b * 2 * L::kSlab);
                        const uint32_t sq = smem_u32(smem + L::kQg + b * 3 * L::kSlab);
                        ok = mbar_wait(&q_full[b], ph, abort_flag, args.status, 0x1E1);
                        // dS^T of the tile was written by the peer: acquire at cluster scope
                        if (ok) ok = mbar_wait_cluster(&ds_full[b], ph, abort_flag, args.status, 0x1E2);
                        // the consumers must have loaded the previous tile's dQ^T out of TMEM
                        if (ok && T > 0) ok = mbar_wait(dq_read, (T - 1) & 1u, abort_flag, args.status, 0x1E3);
                        if (!ok) break;
                        tc_fence_after_sync();
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)      // 16 keys per step
                            mma_ss(tmem_dqn, desc_mn_major(sk + kk * 2048, L::kSlab), desc_mn_major(sds + kk * 2048, L::kSlab),
                                   idesc_dq, kk > 0 ? 1u : 0u);
                        // Rope channels: a 128-row MMA whose rows 64..127 read whatever follows the rope slab in shared
                        // memory (the dS^T buffers); those TMEM lanes are never loaded.
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            mma_ss(tmem_dqr, desc_mn_major(sk + 2 * L::kSlab + kk * 2048, L::kSlab),
                                   desc_mn_major(sds + kk * 2048, L::kSlab), idesc_dq, kk > 0 ? 1u : 0u);
                        mma_commit(dq_full);
                        if (j + 1 == it.n_iter) mma_commit(k_empty);
                        // the first accumulation of an item overwrites dK: the previous item's must be drained
                        if (j == 0 && it.n > 0) ok = mbar_wait(acc_empty, (it.n - 1) & 1u, abort_flag, args.status, 0x1E4);
                        if (!ok) break;
                        tc_fence_after_sync();
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)      // 16 queries per step
                            mma_ss(tmem_dk, desc_k_major(sds + (kk >> 2) * L::kSlab + (kk & 3) * 32),
                                   desc_mn_major(sq + kk * 2048, L::kSlab), idesc_dk, (j > 0 || kk > 0) ? 1u : 0u);
                        mma_commit(&q_empty[b]);
                        mma_commit_to(&ds_free[b], 1u);          // arrives in the score CTA (cluster rank 0)
                        if (j + 1 == it.n_iter) mma_commit(acc_full);
                    }
                }
                if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
            }
        } else {
            const int g = (warp - 2) >> 2;               // query columns [64g, 64g+64) of every dQ^T tile; half of the dK drain
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;         // TMEM lane: channel (dQ^T) or key row (dK)
            const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
            const bool has_rope = quarter < 2;           // lanes 0..63 of the rope accumulator are channels 128..191
            const size_t q_stride = static_cast<size_t>(args.head_count) * 192;
            uint32_t T = 0;
            bool ok = true;
            for (FusedTile it = tile_at(0); it.valid && ok; it = tile_at(it.n + 1)) {
                const int hl = it.head - args.head_begin;
                for (int j = 0; j < it.n_iter && ok; ++j, ++T) {
                    const int q0 = (it.j_begin + j) * 128 + g * 64;
                    ok = mbar_wait_warp(dq_full, T & 1u, abort_flag, args.status, 0x1F0);
                    if (!ok) break;
                    tc_fence_after_sync();
                    // nope channels first; the rope channels' second half is loaded after the nope sums are on their
                    // way, which keeps the live registers under the limit (no more than 96 accumulator words at a time)
                    uint32_t rn[64], rr[32];
                    tmem_ld_x32(tmem_dqn + lane_addr + g * 64, rn);
                    tmem_ld_x32(tmem_dqn + lane_addr + g * 64 + 32, rn + 32);
                    if (has_rope) tmem_ld_x32(tmem_dqr + lane_addr + g * 64, rr);
                    tmem_ld_wait();
                    float* dst = args.dq_acc + (static_cast<size_t>(q0) * args.head_count + hl) * 192 + row;
                    const int n_live = min(64, args.S - q0);       // query rows past the end are not added
                    const bool hl_ok = device_check(hl >= 0 && hl < args.head_count, args.status, 0xE70000u);
                    if (hl_ok) {
#pragma unroll
                        for (int c = 0; c < 64; ++c)
                            if (c < n_live) red_add_f32(dst + c * q_stride, __uint_as_float(rn[c]));
                        if (has_rope) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c < n_live) red_add_f32(dst + c * q_stride + 128, __uint_as_float(rr[c]));
                        }
                    }
                    if (has_rope) {
                        tmem_ld_x32(tmem_dqr + lane_addr + g * 64 + 32, rr);
                        tmem_ld_wait();
                    }
                    tc_fence_before_sync();
                    mbar_arrive(dq_read);
                    if (hl_ok && has_rope) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c + 32 < n_live) red_add_f32(dst + (c + 32) * q_stride + 128, __uint_as_float(rr[c]));
                    }
                }
                if (!ok) break;
                // dK of the finished item: six 32-column chunks (nope 0..3, rope 4..5), three per group
                ok = mbar_wait_warp(acc_full, it.n & 1u, abort_flag, args.status, 0x1F1);
                if (!ok) break;
                tc_fence_after_sync();
                const int t_idx = it.t0 + row;
                const bool valid = t_idx < args.S;
                __nv_bfloat16* dkv_row = args.dkv + static_cast<size_t>(t_idx) * args.h * 256 + it.head * 256;
                float* dkr_row = args.dkpe_acc + static_cast<size_t>(t_idx) * 64;
#pragma unroll 1
                for (int c = g * 3; c < g * 3 + 3; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld_x32(tmem_dk + lane_addr + c * 32, r);
                    tmem_ld_wait();
                    if (!valid) continue;
                    if (!device_check(it.head < args.h && aligned16_dev(dkv_row) && aligned16_dev(dkr_row), args.status, 0xE80000u | c)) continue;
                    if (c >= 4) {
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float4 w = make_float4(__uint_as_float(r[v * 4]) * args.scale, __uint_as_float(r[v * 4 + 1]) * args.scale,
                                                         __uint_as_float(r[v * 4 + 2]) * args.scale, __uint_as_float(r[v * 4 + 3]) * args.scale);
                            atomicAdd(reinterpret_cast<float4*>(dkr_row + (c - 4) * 32) + v, w);
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]) * args.scale, __uint_as_float(r[v * 8 + 1]) * args.scale);
                            w.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]) * args.scale, __uint_as_float(r[v * 8 + 3]) * args.scale);
                            w.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]) * args.scale, __uint_as_float(r[v * 8 + 5]) * args.scale);
                            w.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]) * args.scale, __uint_as_float(r[v * 8 + 7]) * args.scale);
                            reinterpret_cast<uint4*>(dkv_row + c * 32)[v] = w;
                        }
                    }
                }
                __syncwarp();
                tc_fence_before_sync();
                mbar_arrive(acc_empty);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();          // neither CTA leaves while the other may still store into it or signal it
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    clock_probe_end(args.clock_probe);
}

// dq[s, head_begin + i, :] = bf16(scale * dq_acc[s, i, :]); the accumulator is cleared for the next launch.
__global__ void __launch_bounds__(256)
bwd_dq_convert_kernel(float* __restrict__ dq_acc, int S, int h, int head_begin, int head_count, float scale,
                      __nv_bfloat16* __restrict__ dq) {
    grid_launch_dependents();
    grid_dependency_wait();
    const size_t idx = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 8;   // 8 channels per thread
    const size_t row_elems = static_cast<size_t>(head_count) * 192;
    if (idx >= static_cast<size_t>(S) * row_elems) return;
    const size_t s = idx / row_elems, r = idx - s * row_elems;
    float4* src = reinterpret_cast<float4*>(dq_acc + idx);
    const float4 a = src[0], b = src[1];
    src[0] = make_float4(0.f, 0.f, 0.f, 0.f);
    src[1] = make_float4(0.f, 0.f, 0.f, 0.f);
    uint4 w;
    w.x = pack_bf16x2(a.x * scale, a.y * scale);
    w.y = pack_bf16x2(a.z * scale, a.w * scale);
    w.z = pack_bf16x2(b.x * scale, b.y * scale);
    w.w = pack_bf16x2(b.z * scale, b.w * scale);
    *reinterpret_cast<uint4*>(dq + (s * h + head_begin) * 192 + r) = w;
}

}  // namespace laga
