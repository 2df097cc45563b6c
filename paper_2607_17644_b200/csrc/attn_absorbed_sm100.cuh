// Forward attention of the ABSORBED form (Section 3.2, baseline B2): the queries are first carried into
// the latent space, q_abs[s,i,:] = W_uk[i] q_nope[s,i,:] (d_c = 512 wide), scores are taken against the
// gathered latent itself and the shared rope key,
//     s[i,s,t] = scale * ( q_abs[s,i,:] . c_kv[t,:] + q_rope[s,i,:] . k_pe[t,:] ),
// the softmax-weighted sum is accumulated in latent space, o_lat[s,i,:] = sum_t p c_kv[t,:], and only
// then projected to the value dimension by W_uv (a separate GEMM).  No per-head K or V exists; the price
// is a 576-deep score contraction, a 512-wide accumulator per (token, head), and q_abs / o_lat of
// S x h x d_c elements each in memory -- the activation-memory trap of Section 4.3.
//
// The 128 x 512 fp32 accumulator of one query tile alone is all of TMEM, so a CTA owns HALF of the
// latent columns of a (128-query tile, head) item and the scores are computed in both halves' CTAs:
// 2 * (2*576) + 2*512 = 3328 FLOP per (query, key) pair are executed against the form's nominal 2176
// (and the 640 of the explicit form).
//
//   warps 0..3  softmax (one thread per query row): online softmax over 64-key tiles, P written back
//               over the score tile as packed bf16, lazy rescale of the accumulator
//   warp 4      TMA producer: the shared-memory part of Q once, then per key tile the nine 64 x 64
//               slabs of (c_kv || k_pe) in two groups -- the five slabs only the scores read, and the
//               four latent slabs of this CTA's half, which are also the "V" of the second product
//   warp 5      MMA issuer: S = Q K^T (36 k-steps of N = 64: the 16 over this half's latent columns
//               read Q from TMEM, the other 20 from shared memory), O += P V (4 k-steps of N = 256)
// TMEM: [0,256) O half | [256,320) [320,384) two score tiles | [384,512) 256 dims of Q as packed bf16.
#pragma once
#include "attn_fwd_sm100.cuh"
#include "sm100_ptx.cuh"

namespace laga {

struct AttnAbsorbedArgs {
    int S, h;
    float scale_log2;            // softmax_scale * log2(e)
    const __nv_bfloat16* q_abs;  // [S, h, 512]
    __nv_bfloat16* o_lat;        // [S, h, 512]
    float* lse;                  // [S, h]
    unsigned int* status;
};

constexpr int kAbsThreads = 192;
constexpr int kAbsKeys = 64;

struct AttnAbsorbedSmem {
    static constexpr int kQSlab = 128 * 128;                  // 128 query rows x 64 dims
    static constexpr int kKSlab = kAbsKeys * 128;             // 64 keys x 64 dims
    static constexpr int kQ = 0;                              // 5 slabs: the other half's 4 latent slabs, rope
    static constexpr int kK = kQ + 5 * kQSlab;                // 2 stages x 9 slabs (5 score-only, then 4 of this half)
    static constexpr int kBar = kK + 2 * 9 * kKSlab;
    static constexpr int kTotalBytes = kBar + 256;
};
static_assert(AttnAbsorbedSmem::kTotalBytes <= 232448, "absorbed kernel exceeds the 227 KB of shared memory per CTA");

template <bool kCausal>
__global__ void __launch_bounds__(kAbsThreads, 1)
attn_absorbed_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tmap_qabs, const __grid_constant__ CUtensorMap tmap_q,
                               const __grid_constant__ CUtensorMap tmap_ckv, const __grid_constant__ CUtensorMap tmap_kpe,
                               const AttnAbsorbedArgs args) {
    using L = AttnAbsorbedSmem;
    constexpr int BK = kAbsKeys;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* q_full = bars + 0;     // the shared-memory part of Q has landed
    uint64_t* q_ready = bars + 1;    // the TMEM part of Q has been written
    uint64_t* a_full = bars + 2;     // [2]  score-only slabs of the stage
    uint64_t* a_empty = bars + 4;    // [2]
    uint64_t* b_full = bars + 6;     // [2]  this half's latent slabs of the stage
    uint64_t* b_empty = bars + 8;    // [2]
    uint64_t* s_full = bars + 10;    // [2]  score tile T is in TMEM buffer T & 1
    uint64_t* p_full = bars + 12;    // [2]  P of tile T has replaced it
    uint64_t* pv_done = bars + 14;   // [2]  O += P V of tile T has completed
    uint64_t* all_done = bars + 16;
    uint64_t* quiesce_bar = bars + 17;   // abort path only: the MMA lane's last commit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_q_tiles = (args.S + 127) / 128;
    const int q_tile = n_q_tiles - 1 - static_cast<int>(blockIdx.x);   // longest rows first
    const int head = blockIdx.y >> 1, half = blockIdx.y & 1;
    const int q0 = q_tile * 128;
    const int n_keys = kCausal ? min(q0 + 128, args.S) : args.S;
    const int n_kv = (n_keys + BK - 1) / BK;
    const int own_col = half * 256, other_col = (half ^ 1) * 256;      // latent columns of this CTA's half / the other

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1); mbar_init(q_ready, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1);
            mbar_init(&s_full[s], 1); mbar_init(&p_full[s], 128); mbar_init(&pv_done[s], 1);
        }
        mbar_init(all_done, 1);
        mbar_init(quiesce_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_qabs); tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_ckv); tma_prefetch_desc(&tmap_kpe);
        if ((smem_u32(smem) & 1023u) != 0u) {   // the swizzled operand slabs need a 1024-byte aligned base
            abort_flag->value = 1;
        }
    }
    if (warp == 5) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_launch_dependents();
    grid_dependency_wait();          // global memory from here on
    if (threadIdx.x == 0 && abort_flag->value != 0u) atomicCAS(args.status, kStatusOk, kStatusCheck | 0xD3u);   // set-up found the shared memory misaligned
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_s = tmem_base + 256;
    const uint32_t tmem_q = tmem_base + 384;

    if (abort_flag->value != 0u) {
        // misaligned shared memory: nothing was started, fall through to the common exit
    } else if (warp == 4) {
        if (elect_one()) {
            ArmedBarriers armed(bars);
            mbar_arrive_expect_tx(q_full, 5 * L::kQSlab);
            armed.arm(q_full, 0);
            for (int c = 0; c < 4; ++c)
                tma_load_2d_chk(args.status, smem + L::kQ + c * L::kQSlab, &tmap_qabs, q_full, head * 512 + other_col + c * 64, q0);
            tma_load_2d_chk(args.status, smem + L::kQ + 4 * L::kQSlab, &tmap_q, q_full, head * 192 + 128, q0);      // rope band of q
            for (int j = 0; j < n_kv; ++j) {
                const int s = j & 1;
                const uint32_t ph = ((j >> 1) & 1) ^ 1;
                uint8_t* stage = smem + L::kK + s * 9 * L::kKSlab;
                if (!mbar_wait(&a_empty[s], ph, abort_flag, args.status, 0xB0)) break;
                mbar_arrive_expect_tx(&a_full[s], 5 * L::kKSlab);
                armed.arm(&a_full[s], ph ^ 1);
                for (int c = 0; c < 4; ++c)
                    tma_load_2d_chk(args.status, stage + c * L::kKSlab, &tmap_ckv, &a_full[s], other_col + c * 64, j * BK);
                tma_load_2d_chk(args.status, stage + 4 * L::kKSlab, &tmap_kpe, &a_full[s], 0, j * BK);
                if (!mbar_wait(&b_empty[s], ph, abort_flag, args.status, 0xB1)) break;
                mbar_arrive_expect_tx(&b_full[s], 4 * L::kKSlab);
                armed.arm(&b_full[s], ph ^ 1);
                for (int c = 0; c < 4; ++c)
                    tma_load_2d_chk(args.status, stage + (5 + c) * L::kKSlab, &tmap_ckv, &b_full[s], own_col + c * 64, j * BK);
            }
            if (abort_flag->value != 0u) armed.quiesce();
        }
    } else if (warp == 5) {
        if (elect_one()) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, BK, 0, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, 256, 0, 1);
            const uint32_t sq = smem_u32(smem + L::kQ);
            auto issue_qk = [&](int j) -> bool {
                const int s = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                const uint32_t stage = smem_u32(smem + L::kK + s * 9 * L::kKSlab);
                const uint32_t d = tmem_s + s * BK;
                if (!mbar_wait(&a_full[s], ph, abort_flag, args.status, 0xB2)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 20; ++kk)      // the other half's latent dims and the rope band: Q from shared memory
                    mma_ss(d, desc_k_major(sq + (kk >> 2) * L::kQSlab + (kk & 3) * 32),
                           desc_k_major(stage + (kk >> 2) * L::kKSlab + (kk & 3) * 32), idesc_qk, kk > 0 ? 1u : 0u);
                mma_commit(&a_empty[s]);
                if (!mbar_wait(&b_full[s], ph, abort_flag, args.status, 0xB3)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 16; ++kk)      // this half's latent dims: Q from TMEM
                    mma_ts(d, tmem_q + kk * 8, desc_k_major(stage + (5 + (kk >> 2)) * L::kKSlab + (kk & 3) * 32), idesc_qk, 1u);
                mma_commit(&s_full[s]);
                return true;
            };
            bool ok = mbar_wait(q_full, 0, abort_flag, args.status, 0xB4) && mbar_wait(q_ready, 0, abort_flag, args.status, 0xB5);
            if (ok) ok = issue_qk(0);
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j & 1;
                if (j + 1 < n_kv) ok = issue_qk(j + 1);
                if (ok) ok = mbar_wait(&p_full[s], (j >> 1) & 1, abort_flag, args.status, 0xB6);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sv = smem_u32(smem + L::kK + s * 9 * L::kKSlab + 5 * L::kKSlab);
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk)   // A = P: packed bf16, 8 TMEM columns per 16 keys; B = this half's latent slabs
                    mma_ts(tmem_base, tmem_s + s * BK + kk * 8, desc_mn_major(sv + kk * 2048, L::kKSlab), idesc_pv,
                           (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&b_empty[s]);
                mma_commit(&pv_done[s]);
            }
            if (ok) mma_commit(all_done);
            if (abort_flag->value != 0u) { mma_commit(quiesce_bar); mbar_wait_quiesce(quiesce_bar, 0); }
        }
    } else {
        const int row = warp * 32 + lane;             // row inside the tile == TMEM lane
        const int sq_idx = q0 + row;
        const bool valid = sq_idx < args.S;
        const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
        {   // this half's 256 latent dims of the row's q_abs go to TMEM as the A operand of the score MMAs
            const uint4* src = reinterpret_cast<const uint4*>(args.q_abs + (static_cast<size_t>(sq_idx) * args.h + head) * 512 + own_col);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t w[32];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint4 x = valid ? src[c * 8 + v] : make_uint4(0u, 0u, 0u, 0u);
                    w[v * 4] = x.x; w[v * 4 + 1] = x.y; w[v * 4 + 2] = x.z; w[v * 4 + 3] = x.w;
                }
                __syncwarp();
                tmem_st_x32(tmem_q + lane_addr + c * 32, w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(q_ready);
        }
        float m_run = -INFINITY, l_run = 0.f;         // running maximum (scaled, log2 domain) and row sum
        bool ok = true;
        for (int j = 0; j < n_kv; ++j) {
            const int s = j & 1;
            const uint32_t ts = tmem_s + lane_addr + s * BK;
            ok = mbar_wait_warp(&s_full[s], (j >> 1) & 1, abort_flag, args.status, 0xC0);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[BK];
            tmem_ld_x32(ts, sv);
            tmem_ld_x32(ts + 32, sv + 32);
            tmem_ld_wait();
            const int t_last = j * BK + BK - 1;
            if ((kCausal && t_last > q0) || t_last >= args.S) {
#pragma unroll
                for (int c = 0; c < BK; ++c) {
                    const int t = j * BK + c;
                    if ((kCausal && t > sq_idx) || t >= args.S) sv[c] = __float_as_uint(-INFINITY);
                }
            }
            float mxs[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) mxs[e] = fmaxf(__uint_as_float(sv[e]), __uint_as_float(sv[8 + e]));
#pragma unroll
            for (int c = 16; c < BK; c += 16)
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    mxs[e] = fmax3(mxs[e], __uint_as_float(sv[c + e]), __uint_as_float(sv[c + 8 + e]));
            const float mx = fmaxf(fmax3(mxs[0], mxs[1], mxs[2]), fmax3(fmax3(mxs[3], mxs[4], mxs[5]), mxs[6], mxs[7]));
            // Tile 0 holds an unmasked key for every row, so the maximum is finite from there on; a later tile
            // may be masked out for a row altogether (mx = -inf), which leaves it alone and yields P = 0.
            const float m_cand = fmaxf(m_run, mx * args.scale_log2);
            const bool move = (m_cand - m_run) > 8.0f;            // lazy rescale: only when it fell behind by 2^8
            const float m_new = move ? m_cand : m_run;
            const float alpha = move ? fast_exp2(m_run - m_new) : 1.0f;
            m_run = m_new;
            float sums[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            uint32_t pk[BK / 2];
#pragma unroll
            for (int c = 0; c < BK / 2; ++c) {
                const float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * c]), args.scale_log2, -m_new));
                const float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * c + 1]), args.scale_log2, -m_new));
                sums[c & 7] += p0 + p1;
                pk[c] = pack_bf16x2(p0, p1);
            }
            l_run = l_run * alpha + (((sums[0] + sums[1]) + (sums[2] + sums[3])) + ((sums[4] + sums[5]) + (sums[6] + sums[7])));
            if (j > 0 && __any_sync(0xffffffffu, move)) {
                // O must be at rest: P V of the previous tile has finished, P V of this tile waits for p_full below
                ok = mbar_wait_warp(&pv_done[s ^ 1], ((j - 1) >> 1) & 1, abort_flag, args.status, 0xC1);
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    uint32_t o[32];
                    tmem_ld_x32(tmem_base + lane_addr + c * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 32; ++v) o[v] = __float_as_uint(__uint_as_float(o[v]) * alpha);
                    tmem_st_x32(tmem_base + lane_addr + c * 32, o);
                }
            }
            tmem_st_x32(ts, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&p_full[s]);
        }
        if (ok) ok = mbar_wait_warp(all_done, 0, abort_flag, args.status, 0xC2);
        if (ok) {
            tc_fence_after_sync();
            const float inv_l = 1.0f / l_run;
            __nv_bfloat16* dst = args.o_lat + (static_cast<size_t>(sq_idx) * args.h + head) * 512 + own_col;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t o[32];
                __syncwarp();
                tmem_ld_x32(tmem_base + lane_addr + c * 32, o);
                tmem_ld_wait();
                if (valid && device_check(aligned16_dev(dst) && head < args.h, args.status, 0xE60000u | c)) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(o[v * 8 + 0]) * inv_l, __uint_as_float(o[v * 8 + 1]) * inv_l);
                        w.y = pack_bf16x2(__uint_as_float(o[v * 8 + 2]) * inv_l, __uint_as_float(o[v * 8 + 3]) * inv_l);
                        w.z = pack_bf16x2(__uint_as_float(o[v * 8 + 4]) * inv_l, __uint_as_float(o[v * 8 + 5]) * inv_l);
                        w.w = pack_bf16x2(__uint_as_float(o[v * 8 + 6]) * inv_l, __uint_as_float(o[v * 8 + 7]) * inv_l);
                        reinterpret_cast<uint4*>(dst + c * 32)[v] = w;
                    }
                }
            }
            if (valid && half == 0)
                args.lse[static_cast<size_t>(sq_idx) * args.h + head] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace laga
