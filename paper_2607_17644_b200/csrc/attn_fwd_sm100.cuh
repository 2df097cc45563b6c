// Forward attention of Algorithm 1 step 5 for the DeepSeek-V3 head geometry (d_qk = 128 nope + 64
// rope, d_v = 128): O = softmax(scale * q (K_nope || k_pe)^T) V, with LSE, never materialising the
// S x S scores.  K_nope and V are read from the bf16 up-projection KV[S, h*256]; the shared rope
// band k_pe[S, 64] is a separate TMA box, so the 192-wide key is never assembled in memory.
//
// One CTA owns 128 query rows of one head and walks the key tiles (128 keys each).
//   warp 0      TMA producer: K and V tiles, two stages each
//   warp 1      MMA issuer:   S = Q K^T (12 tcgen05.mma of K=16) into one of two TMEM tiles;
//                             O += P V  (8 tcgen05.mma) into a TMEM accumulator.  Both read their A operand
//                             (Q, P) from TMEM: a 128x128 MMA with both operands in shared memory reads
//                             8 KB per 64 clocks, all of the SM's shared-memory bandwidth, and the TMA
//                             writes of the next K/V tile would have to share it.
//   warps 2..5  softmax: one thread per query row; online max / sum in registers; P is written back as
//               packed bf16 over the first 64 columns of the S tile it came from and consumed from
//               there by the second contraction; lazy rescale of O
// The score tile for key tile j+2 reuses the TMEM columns of tile j; it is issued after P_j V_j by the
// same thread, and the tensor pipe executes a thread's MMAs in order, so no extra barrier guards it.
#pragma once
#include "sm100_ptx.cuh"

namespace laga {

struct AttnFwdArgs {
    int S, h;
    float scale_log2;       // softmax_scale * log2(e)
    const __nv_bfloat16* q; // [S, h, 192]
    __nv_bfloat16* out;     // [S, h, 128]
    float* lse;             // [S, h]
    unsigned int* status;
};

struct AttnFwdSmem {
    static constexpr int kSlab = 128 * 128;             // 128 rows x 128 bytes
    static constexpr int kK = 0;                        // 2 stages x 3 slabs (nope lo, nope hi, rope)
    static constexpr int kV = kK + 2 * 3 * kSlab;       // 2 stages x 2 slabs
    static constexpr int kBar = kV + 2 * 2 * kSlab;
    static constexpr int kTotalBytes = kBar + 256 + 1024;
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

template <bool kCausal>
__global__ void __launch_bounds__(192, 1)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                      const AttnFwdArgs args) {
    using L = AttnFwdSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* q_ready = bars + 0;    // the softmax threads have put the Q tile into TMEM
    uint64_t* k_full = bars + 1;     // [2]
    uint64_t* k_empty = bars + 3;    // [2]
    uint64_t* v_full = bars + 5;     // [2]
    uint64_t* v_empty = bars + 7;    // [2]
    uint64_t* s_full = bars + 9;     // [2]
    uint64_t* p_full = bars + 11;
    uint64_t* pv_done = bars + 12;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 13);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_q_tiles = (args.S + 127) / 128;
    const int q_tile = n_q_tiles - 1 - static_cast<int>(blockIdx.x);   // longest rows first
    const int head = blockIdx.y;
    const int q0 = q_tile * 128;
    const int n_kv = kCausal ? q_tile + 1 : n_q_tiles;

    if (threadIdx.x == 0) {
        mbar_init(q_ready, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
            mbar_init(&s_full[s], 1);
        }
        mbar_init(p_full, 128); mbar_init(pv_done, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 256;     // [0,256) two S tiles | [256,384) O | [384,480) Q as packed bf16
    const uint32_t tmem_q = tmem_base + 384;

    if (warp == 0) {
        if (elect_one()) {
            for (int j = 0; j < n_kv; ++j) {
                const int s = j & 1;
                const uint32_t ph_free = ((j >> 1) & 1) ^ 1;
                if (!mbar_wait(&k_empty[s], ph_free, abort_flag, args.status, 0x10)) break;
                uint8_t* dk = smem + L::kK + s * 3 * L::kSlab;
                mbar_arrive_expect_tx(&k_full[s], 3 * L::kSlab);
                tma_load_2d(dk, &tmap_kv, &k_full[s], head * 256, j * 128);
                tma_load_2d(dk + L::kSlab, &tmap_kv, &k_full[s], head * 256 + 64, j * 128);
                tma_load_2d(dk + 2 * L::kSlab, &tmap_kpe, &k_full[s], 0, j * 128);
                if (!mbar_wait(&v_empty[s], ph_free, abort_flag, args.status, 0x11)) break;
                uint8_t* dv = smem + L::kV + s * 2 * L::kSlab;
                mbar_arrive_expect_tx(&v_full[s], 2 * L::kSlab);
                tma_load_2d(dv, &tmap_kv, &v_full[s], head * 256 + 128, j * 128);
                tma_load_2d(dv + L::kSlab, &tmap_kv, &v_full[s], head * 256 + 192, j * 128);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, 0, 1);
            auto issue_qk = [&](int j) -> bool {
                const int s = j & 1;
                if (!mbar_wait(&k_full[s], (j >> 1) & 1, abort_flag, args.status, 0x23)) return false;
                tc_fence_after_sync();
                const uint32_t sk = smem_u32(smem + L::kK + s * 3 * L::kSlab);
#pragma unroll
                for (int kk = 0; kk < 12; ++kk) {
                    const uint32_t off = (kk >> 2) * L::kSlab + (kk & 3) * 32;
                    mma_ts(tmem_base + s * 128, tmem_q + kk * 8, desc_k_major(sk + off), idesc_qk, kk > 0 ? 1u : 0u);
                }
                mma_commit(&k_empty[s]);
                mma_commit(&s_full[s]);
                return true;
            };
            bool ok = mbar_wait(q_ready, 0, abort_flag, args.status, 0x22);
            tc_fence_after_sync();
            if (ok) ok = issue_qk(0);
            if (ok && n_kv > 1) ok = issue_qk(1);
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j & 1;
                ok = mbar_wait(&v_full[s], (j >> 1) & 1, abort_flag, args.status, 0x20) &&
                     mbar_wait(p_full, j & 1, abort_flag, args.status, 0x21);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sv = smem_u32(smem + L::kV + s * 2 * L::kSlab);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)   // A = P_j: packed bf16, 8 TMEM columns per 16 keys
                    mma_ts(tmem_o, tmem_base + s * 128 + kk * 8, desc_mn_major(sv + kk * 2048, L::kSlab), idesc_pv,
                           (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&v_empty[s]);
                mma_commit(pv_done);
                if (j + 2 < n_kv) ok = issue_qk(j + 2);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;          // row inside the tile == TMEM lane
        const int sq_idx = q0 + row;                  // global query index
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        {   // this thread's query row (192 bf16 = 96 packed words) goes to TMEM once, as the A operand of S
            const bool q_valid = sq_idx < args.S;
            const uint4* src = reinterpret_cast<const uint4*>(args.q + (static_cast<size_t>(sq_idx) * args.h + head) * 192);
#pragma unroll 1
            for (int c = 0; c < 3; ++c) {
                uint32_t w[32];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint4 x = q_valid ? src[c * 8 + v] : make_uint4(0u, 0u, 0u, 0u);
                    w[v * 4] = x.x; w[v * 4 + 1] = x.y; w[v * 4 + 2] = x.z; w[v * 4 + 3] = x.w;
                }
                __syncwarp();
                tmem_st_x32(tmem_q + lane_addr + c * 32, w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(q_ready);
        }
        float m_run = -INFINITY, l_run = 0.f;         // running max (scaled, log2 domain) and sum
        bool ok = true;
        for (int j = 0; j < n_kv; ++j) {
            const int s = j & 1;
            ok = mbar_wait_warp(&s_full[s], (j >> 1) & 1, abort_flag, args.status, 0x30);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_x32(tmem_base + lane_addr + s * 128 + c * 32, sv + c * 32);
            tmem_ld_wait();

            const bool edge = (j == n_kv - 1);
            if (edge) {
#pragma unroll
                for (int c = 0; c < 128; ++c) {
                    const int t = j * 128 + c;
                    if ((kCausal && t > sq_idx) || t >= args.S) sv[c] = __float_as_uint(-INFINITY);
                }
            }
            // eight independent chains: a single warp per scheduler cannot hide a 128-deep dependency
            // (three-input max: two elements per instruction)
            float mxs[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) mxs[e] = fmaxf(__uint_as_float(sv[e]), __uint_as_float(sv[8 + e]));
#pragma unroll
            for (int c = 16; c < 128; c += 16)
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    mxs[e] = fmax3(mxs[e], __uint_as_float(sv[c + e]), __uint_as_float(sv[c + 8 + e]));
            const float mx = fmaxf(fmax3(mxs[0], mxs[1], mxs[2]), fmax3(fmax3(mxs[3], mxs[4], mxs[5]), mxs[6], mxs[7]));
            const float m_new = fmaxf(m_run, mx * args.scale_log2);
            // Lazy rescale: keep the old reference max unless it fell behind by more than 2^8.
            const bool move = (m_new - m_run) > 8.0f;
            const float alpha = move ? fast_exp2(m_run - m_new) : 1.0f;
            if (move) m_run = m_new;
            float sums[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            uint32_t pk[64];
#pragma unroll
            for (int c = 0; c < 64; ++c) {
                const float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * c]), args.scale_log2, -m_run));
                const float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * c + 1]), args.scale_log2, -m_run));
                sums[c & 7] += p0 + p1;
                pk[c] = pack_bf16x2(p0, p1);
            }
            const float sum = ((sums[0] + sums[1]) + (sums[2] + sums[3])) + ((sums[4] + sums[5]) + (sums[6] + sums[7]));
            l_run = l_run * alpha + sum;

            if (j > 0 && __any_sync(0xffffffffu, move)) {
                // O must be at rest: P_{j-1} V_{j-1} finished, P_j V_j not issued before p_full below.
                ok = mbar_wait_warp(pv_done, (j - 1) & 1, abort_flag, args.status, 0x31);
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
            tmem_st_x32(tmem_base + lane_addr + s * 128, pk);
            tmem_st_x32(tmem_base + lane_addr + s * 128 + 32, pk + 32);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(p_full);
        }
        if (ok) ok = mbar_wait_warp(pv_done, (n_kv - 1) & 1, abort_flag, args.status, 0x32);
        if (ok) {
            tc_fence_after_sync();
            const float inv_l = 1.0f / l_run;
            const bool valid = sq_idx < args.S;
            __nv_bfloat16* dst = args.out + (static_cast<size_t>(sq_idx) * args.h + head) * 128;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                __syncwarp();
                tmem_ld_x32(tmem_o + lane_addr + c * 32, o);
                tmem_ld_wait();
                if (valid) {
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
            if (valid)
                args.lse[static_cast<size_t>(sq_idx) * args.h + head] = (m_run + log2f(l_run)) * 0.6931471805599453f;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace laga
