// Forward attention of Algorithm 1 step 5 for the DeepSeek-V3 head geometry (d_qk = 128 nope + 64
// rope, d_v = 128): O = softmax(scale * q (K_nope || k_pe)^T) V, with LSE, never materialising the
// S x S scores.  K_nope and V are read from the bf16 up-projection KV[S, h*256]; the shared rope
// band k_pe[S, 64] is a separate TMA box, so the 192-wide key is never assembled in memory.
//
// One CTA owns 128 query rows of one head and walks the key tiles (96 keys each).
//   warps 0..3  softmax warpgroup 0: even key tiles      one thread per query row in each group; the
//   warps 4..7  softmax warpgroup 1: odd key tiles       exponentials of one group's tile run beside
//                                                        the row maximum / load / store phases of the other's
//   warp 8      TMA producer: K tiles, three stages
//   warp 9      MMA issuer:   S = Q K^T (12 tcgen05.mma of K=16, N=96) into one of three TMEM tiles;
//                             O += P V (6 tcgen05.mma of N=128).  Both read their A operand (Q, P) from TMEM:
//                             an MMA with both operands in shared memory is bound by shared-memory
//                             bandwidth (128 B/clk).
//   warp 10     TMA producer: V tiles, three stages; ahead of each item's tiles the item's query tile as three ring entries
// Why 96 keys: the Q tile (96 columns of packed bf16), the O accumulator (128) and THREE score tiles
// (3 x 96) fill the 512 TMEM columns exactly.  With three score tiles the tensor pipe computes S_{j+3}
// while the two groups work on tiles j+1 and j+2, so neither side waits for the other; with 128-key
// tiles only two fit and the chain S -> softmax -> P V -> next S on the same columns sets the pace.
// The two groups share one running reference maximum per row (a word of shared memory handed from
// tile to tile through the max_done barriers: only the short row-maximum phase is serial, the
// exponentials are not) and therefore one O accumulator; each keeps its own partial row sum, brought
// to the common reference at the end.  P is written back as packed bf16 over the first 48 columns of
// the S tile it came from.  The score tile for key tile j+3 reuses the TMEM columns of tile j; it is
// issued after P_j V_j by the same thread, and the tensor pipe executes a thread's MMAs in order, so
// no extra barrier guards it.
#pragma once
#include "sm100_ptx.cuh"
#include "work_sched.cuh"

namespace laga {

struct AttnFwdArgs {
    int S, h;
    float scale_log2;       // softmax_scale * log2(e)
    const __nv_bfloat16* q; // [S, h, 192]
    __nv_bfloat16* out;     // [S, h, 128]
    float* lse;             // [S, h]
    unsigned int* status;
    WorkSchedule sched;     // items = (128-query tile, head); rank 0 = the last query tile (most keys)
    ClockProbe* clock_probe;   // may be nullptr
};

constexpr int kFwdThreads = 352;
constexpr int kFwdKeys = 96;     // keys per tile
constexpr int kFwdStages = 3;

struct AttnFwdSmem {
    static constexpr int kSlab = kFwdKeys * 128;                 // 96 rows x 128 bytes
    static constexpr int kK = 0;                                 // stages x 3 slabs (nope lo, nope hi, rope)
    static constexpr int kV = kK + kFwdStages * 3 * kSlab;       // stages x 2 slabs
    static constexpr int kMref = kV + kFwdStages * 2 * kSlab;    // 128 floats: the rows' reference maxima
    static constexpr int kLsum = kMref + 512;                    // 2 items x 2 groups x 128 floats: row sums
    static constexpr int kBar = kLsum + 2048;
    static constexpr int kTotalBytes = kBar + 512;
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Persistent: one CTA per SM takes (query tile, head) items from the work counter.  The K, V and
// score-tile rings and the alternation of the two softmax groups run on a tile count that continues
// across items, so the producers prefetch the next item's first key tiles under the current item's
// last ones; between items, the next query tile comes through the V ring and the MMA lane copies it
// to TMEM (tcgen05.cp) while the softmax groups drain the finished O, so the next item's first score
// MMAs run under the drain.
template <bool kCausal>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                      const __grid_constant__ CUtensorMap tmap_kpe, const AttnFwdArgs args) {
    using L = AttnFwdSmem;
    constexpr int BK = kFwdKeys;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* k_full = bars + 1;     // [3]
    uint64_t* k_empty = bars + 4;    // [3]
    uint64_t* v_full = bars + 7;     // [3]
    uint64_t* v_empty = bars + 10;   // [3]
    uint64_t* s_full = bars + 13;    // [3]  S of tile T is in TMEM buffer T % 3
    // One barrier per SCORE BUFFER, not per softmax group: with three score tiles in flight a group can have
    // delivered P of tile T+1 and of tile T+3 before the MMA lane (held up, say, by a late V stage) has looked
    // at the first; a per-group barrier would then be two phases ahead of its waiter, whose parity test can
    // no longer tell "done" from "not yet" (it waits for ever).  A buffer cannot be refilled before its
    // previous P was consumed, so a per-buffer barrier never runs ahead.
    uint64_t* p_full = bars + 16;    // [3]  P of tile T has replaced S in buffer T % 3
    uint64_t* pv_done = bars + 19;   // [2]  P V of a tile of group g has completed
    uint64_t* max_done = bars + 21;  // [2]  group g has published the reference maxima of its tile
    uint64_t* all_done = bars + 23;  // every MMA of the item has completed
    uint64_t* l_ready = bars + 24;   // both groups have stored their row sums
    uint64_t* o_empty = bars + 25;   // both groups have drained O
    ItemRing ring{bars + 26, bars + 28, reinterpret_cast<volatile int*>(bars + 30)};
    uint64_t* quiesce_bar = bars + 31;   // abort path only: the MMA lane's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 32);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);
    float* mref = reinterpret_cast<float*>(smem + L::kMref);
    float* lsum = reinterpret_cast<float*>(smem + L::kLsum);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 3; ++s) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); mbar_init(&s_full[s], 1);
            mbar_init(&p_full[s], 128);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&pv_done[s], 1); mbar_init(&max_done[s], 128);
            mbar_init(&ring.full[s], 1); mbar_init(&ring.empty[s], 10);
        }
        mbar_init(all_done, 1);
        mbar_init(l_ready, 256);
        mbar_init(o_empty, 256);
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
        if ((smem_u32(smem) & 1023u) != 0u) {   // the swizzled operand slabs need a 1024-byte aligned base
            abort_flag->value = 1;
        }
    }
    if (warp == 9) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();          // set-up above overlaps the previous kernel's tail; global memory from here on
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD2u);   // set-up found the shared memory misaligned
    clock_probe_begin(args.clock_probe);
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 3 * BK;       // [0,288) three S tiles | [288,416) O | [416,512) Q as packed bf16
    const uint32_t tmem_q = tmem_o + 128;
    // q0 and every key index are relative to the item's sequence; row_base is the sequence's first row in the
    // packed tensors and S_seq its length (0 and S for a single sequence).
    auto item_geometry = [&](int item, int& q0, int& head, int& n_kv, int& row_base, int& S_seq) {
        int rank;
        decode_item(args.sched, item, rank, head);
        const SeqTile st = seq_tile(args.sched, rank, args.S, true);    // longest rows first
        q0 = st.tile * 128;
        row_base = st.seq_start;
        S_seq = st.seq_len;
        const int n_keys = kCausal ? min(q0 + 128, S_seq) : S_seq;      // keys any row of this tile attends to
        n_kv = (n_keys + BK - 1) / BK;
    };

    if (abort_flag->value != 0u) {
        // misaligned shared memory: nothing was started, fall through to the common exit
    } else if (warp == 8) {
        // K and V have producers of their own: the score MMAs run up to three tiles ahead of the P V MMAs,
        // and a single thread waiting for a V stage would hold back the K tile the tensor pipe needs next.
        if (elect_one()) {
            uint32_t T = 0;
            bool ok = true;
            ArmedBarriers armed(bars);
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_publish(ring, args.sched, n, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int q0, head, n_kv, row_base, S_seq;
                item_geometry(item, q0, head, n_kv, row_base, S_seq);
                for (int j = 0; j < n_kv; ++j, ++T) {
                    const uint32_t s = T % kFwdStages;
                    ok = mbar_wait(&k_empty[s], ((T / kFwdStages) & 1u) ^ 1u, abort_flag, args.status, 0x10);
                    if (!ok) break;
                    uint8_t* dk = smem + L::kK + s * 3 * L::kSlab;
                    mbar_arrive_expect_tx(&k_full[s], 3 * L::kSlab);
                    armed.arm(&k_full[s], (T / kFwdStages) & 1u);
                    tma_load_2d_chk(args.status, dk, &tmap_kv, &k_full[s], head * 256, row_base + j * BK);
                    tma_load_2d_chk(args.status, dk + L::kSlab, &tmap_kv, &k_full[s], head * 256 + 64, row_base + j * BK);
                    tma_load_2d_chk(args.status, dk + 2 * L::kSlab, &tmap_kpe, &k_full[s], 0, row_base + j * BK);
                }
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 10) {
        if (elect_one()) {
            uint32_t T = 0;
            bool ok = true;
            ArmedBarriers armed(bars);
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_read(ring, n, true, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int q0, head, n_kv, row_base, S_seq;
                item_geometry(item, q0, head, n_kv, row_base, S_seq);
                // The item's query tile travels through the V ring ahead of the item's value tiles: three slabs of
                // 128 rows x 64 elements, one ring entry each (a stage holds 24 KB, a slab is 16 KB).  Three entries
                // are one turn of the ring, so the value tiles keep their stages; every item shifts the barriers'
                // phases by one.  The MMA lane copies the slabs to TMEM (tcgen05.cp): no thread's load/store unit
                // sees the tile -- a lane reading its own row touches 32 lines per instruction, and done that way
                // the staging cost four to seven thousand clocks per item on the softmax warps.
                for (uint32_t c = 0; c < 3u && ok; ++c) {
                    const uint32_t Tc = T + c, s = Tc % kFwdStages, ph = ((Tc / kFwdStages) + n) & 1u;
                    ok = mbar_wait(&v_empty[s], ph ^ 1u, abort_flag, args.status, 0x12);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&v_full[s], 128 * 128);
                    armed.arm(&v_full[s], ph);
                    tma_load_2d_chk(args.status, smem + L::kV + s * 2 * L::kSlab, &tmap_q, &v_full[s], head * 192 + static_cast<int>(c) * 64,
                                    row_base + q0);      // rows past the tensor's end read as zero
                }
                if (!ok) break;
                for (int j = 0; j < n_kv; ++j, ++T) {
                    const uint32_t s = T % kFwdStages, phv = ((T / kFwdStages) + n + 1u) & 1u;
                    ok = mbar_wait(&v_empty[s], phv ^ 1u, abort_flag, args.status, 0x11);
                    if (!ok) break;
                    uint8_t* dv = smem + L::kV + s * 2 * L::kSlab;
                    mbar_arrive_expect_tx(&v_full[s], 2 * L::kSlab);
                    armed.arm(&v_full[s], phv);
                    tma_load_2d_chk(args.status, dv, &tmap_kv, &v_full[s], head * 256 + 128, row_base + j * BK);
                    tma_load_2d_chk(args.status, dv + L::kSlab, &tmap_kv, &v_full[s], head * 256 + 192, row_base + j * BK);
                }
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 9) {
        if (elect_one()) {
            // tcgen05.mma issue is close to synchronous with the tensor pipe (about one MMA of queue), so
            // whatever else this thread does is time the pipe idles: an mbarrier wait costs some 90 clocks
            // even when the barrier is already complete.  Each barrier is therefore probed BEFORE the
            // preceding batch of MMAs is issued and the answer read after it: the probe's latency passes
            // while the MMAs block, and the bounded wait runs only when the probe came back false.
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, BK, 0, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, 0, 1);
            const uint64_t desc_k0 = desc_k_major(smem_u32(smem + L::kK));
            const uint64_t desc_v0 = desc_mn_major(smem_u32(smem + L::kV), L::kSlab);
            const uint32_t k_lo0 = static_cast<uint32_t>(desc_k0), k_hi = static_cast<uint32_t>(desc_k0 >> 32);
            const uint32_t v_lo0 = static_cast<uint32_t>(desc_v0), v_hi = static_cast<uint32_t>(desc_v0 >> 32);
            constexpr uint32_t kKStageLo = (3 * L::kSlab) >> 4, kVStageLo = (2 * L::kSlab) >> 4;
            const uint32_t bars_a = smem_u32(bars);
            auto qk_mmas = [&](uint32_t T) {
                const uint32_t s = T % kFwdStages;
                mma_ts_chain_qk96_head(tmem_base + s * BK, tmem_q, k_lo0 + s * kKStageLo, k_hi, idesc_qk);
                mma_ts_chain_qk96_tail(tmem_base + s * BK, tmem_q, k_lo0 + s * kKStageLo, k_hi, idesc_qk, bars_a + (4u + s) * 8u, bars_a + (13u + s) * 8u);
            };
            uint32_t T0 = 0;
            bool ok = true;
            for (uint32_t n = 0; ok; ++n) {
                const int item = ring_read(ring, n, true, abort_flag, args.status, ok);
                if (!ok || item < 0) break;
                int q0, head, n_kv, row_base, S_seq;
                item_geometry(item, q0, head, n_kv, row_base, S_seq);
                // The item's query tile: three entries of the V ring, copied to TMEM as the A operand of S.  (Every
                // MMA that read the previous tile has completed: the previous item's last P V was issued after the
                // softmax of its last score tile.)
                for (uint32_t c = 0; c < 3u && ok; ++c) {
                    const uint32_t Tc = T0 + c, s = Tc % kFwdStages;
                    ok = mbar_wait(&v_full[s], ((Tc / kFwdStages) + n) & 1u, abort_flag, args.status, 0x22);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t src = smem_u32(smem + L::kV + s * 2 * L::kSlab);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) tmem_cp_128x256b(tmem_q + c * 32 + kk * 8, desc_k_major(src + kk * 32));
                    mma_commit(&v_empty[s]);
                }
                const uint32_t vflip = (n + 1u) & 1u;     // phase shift of the V ring's barriers for this item's tiles
                for (int j = 0; j < 3 && j < n_kv && ok; ++j) {
                    const uint32_t T = T0 + j;
                    ok = mbar_wait(&k_full[T % kFwdStages], (T / kFwdStages) & 1u, abort_flag, args.status, 0x23);
                    tc_fence_after_sync();
                    if (ok) qk_mmas(T);
                }
                // the item's first P V overwrites O: the previous item's must have been drained
                if (ok && n > 0) ok = mbar_wait(o_empty, (n - 1) & 1u, abort_flag, args.status, 0x24);
                bool v_ok = false, p_ok = false;      // probes of v_full / p_full for tile j
                for (int j = 0; j < n_kv && ok; ++j) {
                    const uint32_t T = T0 + j;
                    const uint32_t s = T % kFwdStages, g = T & 1u;
                    const uint32_t ph = (T / kFwdStages) & 1u;
                    if (!v_ok) ok = mbar_wait(&v_full[s], ph ^ vflip, abort_flag, args.status, 0x20);
                    if (ok && !p_ok) ok = mbar_wait(&p_full[s], ph, abort_flag, args.status, 0x21);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const bool more = j + 3 < n_kv;
                    const bool k_ok = more && mbar_try_wait(&k_full[s], ph ^ 1u);   // K of tile T+3 lands in the stage tile T left
                    mma_ts_chain_pv96_head(tmem_o, tmem_base + s * BK, v_lo0 + s * kVStageLo, v_hi, idesc_pv, static_cast<uint32_t>(j));
                    mma_ts_chain_pv96_tail(tmem_o, tmem_base + s * BK, v_lo0 + s * kVStageLo, v_hi, idesc_pv, bars_a + (10u + s) * 8u, bars_a + (19u + g) * 8u);
                    v_ok = p_ok = false;
                    if (more) {
                        if (!k_ok) ok = mbar_wait(&k_full[s], ph ^ 1u, abort_flag, args.status, 0x23);
                        if (!ok) break;
                        tc_fence_after_sync();
                        v_ok = mbar_try_wait(&v_full[(T + 1) % kFwdStages], (((T + 1) / kFwdStages) & 1u) ^ vflip);
                        p_ok = mbar_try_wait(&p_full[(T + 1) % kFwdStages], ((T + 1) / kFwdStages) & 1u);
                        qk_mmas(T + 3);
                    }
                }
                if (ok) mma_commit(all_done);
                T0 += static_cast<uint32_t>(n_kv);
            }
            if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        const int g = warp >> 2;                      // softmax warpgroup: tiles whose running count has parity g
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;          // row inside the tile == TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        auto read_item = [&](uint32_t n, bool& ok) -> int {
            ok = mbar_wait_warp(&ring.full[n & 1u], (n >> 1) & 1u, abort_flag, args.status, 0xA1);
            if (!ok) return -1;
            const int it = ring.item[n & 1u];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ring.empty[n & 1u]);
            return it;
        };
        // O of a finished item (all of its MMAs are known complete): each group drains half of the columns
        // (sq_idx: the row in the packed tensors; valid: it lies inside its sequence)
        auto drain = [&](int sq_idx, bool valid, int head, float m_fin, float l_run) {
            tc_fence_after_sync();
            const float inv_l = 1.0f / l_run;
            __nv_bfloat16* dst = args.out + (static_cast<size_t>(sq_idx) * args.h + head) * 128;
            const bool wide = aligned32_dev(args.out);
#pragma unroll 1
            for (int c = 2 * g; c < 2 * g + 2; ++c) {
                uint32_t o[32];
                __syncwarp();
                tmem_ld_x32(tmem_o + lane_addr + c * 32, o);
                tmem_ld_wait();
                if (valid && device_check(aligned16_dev(dst) && head < args.h && sq_idx >= 0, args.status, 0xE30000u | c)) {
                    uint32_t w[16];
#pragma unroll
                    for (int v = 0; v < 16; ++v) w[v] = pack_bf16x2(__uint_as_float(o[2 * v]) * inv_l, __uint_as_float(o[2 * v + 1]) * inv_l);
                    if (wide) {          // two 32-byte stores per 32-column chunk (rows are 256 bytes)
                        st_global_v8(dst + c * 32, w);
                        st_global_v8(dst + c * 32 + 16, w + 8);
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            reinterpret_cast<uint4*>(dst + c * 32)[v] = make_uint4(w[v * 4], w[v * 4 + 1], w[v * 4 + 2], w[v * 4 + 3]);
                    }
                }
            }
            if (valid && g == 0)
                args.lse[static_cast<size_t>(sq_idx) * args.h + head] = (m_fin + log2f(l_run)) * 0.6931471805599453f;
            __syncwarp();
            tc_fence_before_sync();
            mbar_arrive(o_empty);
        };
        uint32_t T0 = 0;
        bool ok = true;
        int item = read_item(0, ok);
        int prev_sq_idx = 0, prev_head = 0;
        bool prev_valid = false;
        float prev_m_fin = 0.f, prev_l_run = 1.f;
        for (uint32_t n = 0; ok && item >= 0; ++n) {
            int q0, head, n_kv, row_base, S_seq;
            item_geometry(item, q0, head, n_kv, row_base, S_seq);
            const int sq_idx = q0 + row;              // query index within the sequence
            if (n > 0) drain(prev_sq_idx, prev_valid, prev_head, prev_m_fin, prev_l_run);
            float m_mine = -INFINITY;                     // reference max (scaled, log2 domain) l_part refers to
            float l_part = 0.f;                           // this group's part of the row sum
            for (int j = 0; j < n_kv; ++j) {
                const uint32_t T = T0 + j;
                if ((T & 1u) != static_cast<uint32_t>(g)) continue;
                const uint32_t b = T % kFwdStages;
                const uint32_t tmem_s = tmem_base + lane_addr + b * BK;
                ok = mbar_wait_warp(&s_full[b], (T / kFwdStages) & 1u, abort_flag, args.status, 0x30);
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t sv[BK];
#pragma unroll
                for (int c = 0; c < BK / 32; ++c) tmem_ld_x32(tmem_s + c * 32, sv + c * 32);
                tmem_ld_wait();

                const int t_last = j * BK + BK - 1;
                if ((kCausal && t_last > q0) || t_last >= S_seq) {   // the causal edge can cross two tiles
#pragma unroll
                    for (int c = 0; c < BK; ++c) {
                        const int t = j * BK + c;
                        if ((kCausal && t > sq_idx) || t >= S_seq) sv[c] = __float_as_uint(-INFINITY);
                    }
                }
                // eight independent chains (three-input max: two elements per instruction)
                float mxs[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) mxs[e] = fmaxf(__uint_as_float(sv[e]), __uint_as_float(sv[8 + e]));
#pragma unroll
                for (int c = 16; c < BK; c += 16)
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        mxs[e] = fmax3(mxs[e], __uint_as_float(sv[c + e]), __uint_as_float(sv[c + 8 + e]));
                const float mx = fmaxf(fmax3(mxs[0], mxs[1], mxs[2]), fmax3(fmax3(mxs[3], mxs[4], mxs[5]), mxs[6], mxs[7]));

                // The reference maximum as the other group left it after the item's previous tile.  The item's
                // first tile holds an unmasked key for every row, so the reference is finite from there on; a
                // later tile may be masked out for a row altogether (mx = -inf), which leaves the reference alone
                // and yields P = 0.
                float m_old = -INFINITY;
                if (j > 0) {
                    ok = mbar_wait_warp(&max_done[g ^ 1], ((T - 1) >> 1) & 1u, abort_flag, args.status, 0x33);
                    if (!ok) break;
                    m_old = mref[row];
                }
                const float m_cand = fmaxf(m_old, mx * args.scale_log2);
                // Lazy rescale: keep the old reference unless it fell behind by more than 2^8.
                const bool move = (m_cand - m_old) > 8.0f;
                const float m_new = move ? m_cand : m_old;
                if (move) mref[row] = m_new;
                mbar_arrive(&max_done[g]);
                const float alpha = move ? fast_exp2(m_old - m_new) : 1.0f;               // for O (all earlier tiles)
                const float beta = (m_mine == m_new) ? 1.0f : fast_exp2(m_mine - m_new);   // for this group's sum
                m_mine = m_new;

                float sums[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                uint32_t pk[BK / 2];
#pragma unroll
                for (int c = 0; c < BK / 2; ++c) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * c]), args.scale_log2, -m_new));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * c + 1]), args.scale_log2, -m_new));
                    sums[c & 7] += p0 + p1;
                    pk[c] = pack_bf16x2(p0, p1);
                }
                const float sum = ((sums[0] + sums[1]) + (sums[2] + sums[3])) + ((sums[4] + sums[5]) + (sums[6] + sums[7]));
                l_part = l_part * beta + sum;

                if (j > 0 && __any_sync(0xffffffffu, move)) {
                    // O must be at rest: P V of the previous tile finished (the previous phase of its barrier, tile
                    // T-3, is known complete because S of this tile was issued after it), P V of this tile is not
                    // issued before p_full below.
                    ok = mbar_wait_warp(&pv_done[g ^ 1], ((T - 1) >> 1) & 1u, abort_flag, args.status, 0x31);
                    if (!ok) break;
                    tc_fence_after_sync();
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[32];
                        tmem_ld_x32(tmem_o + lane_addr + c * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int v = 0; v < 32; ++v) o[v] = __float_as_uint(__uint_as_float(o[v]) * alpha);
                        tmem_st_x32(tmem_o + lane_addr + c * 32, o);
                    }
                }
                tmem_st_x32(tmem_s, pk);
                tmem_st_x16(tmem_s + 32, pk + 32);
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(&p_full[b]);
            }
            if (!ok) break;
            // Bring this group's sum to the final reference (set by the owner of the item's last tile) and add
            // the two groups' sums.
            const uint32_t last = T0 + static_cast<uint32_t>(n_kv) - 1u;
            if ((last & 1u) != static_cast<uint32_t>(g))
                ok = mbar_wait_warp(&max_done[g ^ 1], (last >> 1) & 1u, abort_flag, args.status, 0x34);
            if (!ok) break;
            const float m_fin = mref[row];
            float* lsum_n = lsum + (n & 1u) * 256;
            lsum_n[g * 128 + row] = l_part * ((m_mine == m_fin) ? 1.0f : fast_exp2(m_mine - m_fin));
            mbar_arrive(l_ready);
            ok = mbar_wait_warp(l_ready, n & 1u, abort_flag, args.status, 0x35);
            if (!ok) break;
            prev_l_run = lsum_n[row] + lsum_n[128 + row];
            prev_m_fin = m_fin;
            prev_sq_idx = row_base + sq_idx;
            prev_valid = sq_idx < S_seq;
            prev_head = head;
            ok = mbar_wait_warp(all_done, n & 1u, abort_flag, args.status, 0x32);
            if (!ok) break;
            T0 += static_cast<uint32_t>(n_kv);
            item = read_item(n + 1, ok);
            if (ok && item < 0) drain(prev_sq_idx, prev_valid, prev_head, prev_m_fin, prev_l_run);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    clock_probe_end(args.clock_probe);
}

}  // namespace laga
