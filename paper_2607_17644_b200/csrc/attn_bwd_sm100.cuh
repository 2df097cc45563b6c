// Backward of Algorithm 1 step 5 (Section 5.2: the chain rule through the softmax attention) for
// the DeepSeek-V3 head geometry, as two tcgen05 kernels that recompute P from the saved LSE:
//
//   attn_bwd_dkv  one CTA per (128-key tile, head), sweeping the 64-row query tiles that attend to it:
//                 S^T = K Q^T, dP^T = V dO^T, P^T = exp(scale S^T - LSE), dS^T = P^T (dP^T - delta),
//                 dV += P^T dO, dK += dS^T Q  (dK 192 wide: 128 nope columns + 64 rope columns).
//                 TMEM lanes are keys, so LSE and delta are per-column vectors staged in shared memory.
//   attn_bwd_dq   one CTA per (128-query tile, head), sweeping 64-key tiles:
//                 S = Q K^T, dP = dO V^T, dS = P (dP - delta), dQ += dS K.  TMEM lanes are queries.
//
// Both read K_nope / V from the recomputed bf16 up-projection KV[S, h*256] and the shared rope band
// from k_pe[S, 64]; both keep every accumulator in TMEM and never materialise S x S.
#pragma once
#include "attn_fwd_sm100.cuh"
#include "sm100_ptx.cuh"

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
// past the end of the sequence produce P = 0.
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                 const float* __restrict__ lse, int S, int h, int S_pad, float* __restrict__ stat_l2,
                 float* __restrict__ stat_delta) {
    const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp_global >= S_pad * h) return;
    const int s = warp_global / h, i = warp_global % h;
    if (s >= S) {
        if (lane == 0) {
            stat_l2[static_cast<size_t>(i) * S_pad + s] = INFINITY;
            stat_delta[static_cast<size_t>(i) * S_pad + s] = 0.f;
        }
        return;
    }
    const size_t base = (static_cast<size_t>(s) * h + i) * 128 + lane * 4;
    const uint2 a = *reinterpret_cast<const uint2*>(out + base);
    const uint2 b = *reinterpret_cast<const uint2*>(dout + base);
    const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&b);
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const float2 x = __bfloat1622float2(a2[k]), y = __bfloat1622float2(b2[k]);
        acc = fmaf(x.x, y.x, acc);
        acc = fmaf(x.y, y.y, acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) {
        stat_l2[static_cast<size_t>(i) * S_pad + s] = lse[static_cast<size_t>(s) * h + i] * 1.4426950408889634f;
        stat_delta[static_cast<size_t>(i) * S_pad + s] = acc;
    }
}

// dk_pe[t, r] = sum over heads of the per-head rope-column key gradients (Section 5.3: the rope band
// is shared by every head, so its gradient is the sum over the head shard).
__global__ void __launch_bounds__(256)
bwd_dkpe_reduce_kernel(const float* __restrict__ dk_rope, int S, int h, __nv_bfloat16* __restrict__ dk_pe) {
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t n = static_cast<size_t>(S) * 64;
    if (idx >= n) return;
    float acc = 0.f;
    for (int i = 0; i < h; ++i) acc += dk_rope[static_cast<size_t>(i) * n + idx];
    dk_pe[idx] = __float2bfloat16_rn(acc);
}

// ================================================================================================
// dK / dV kernel
// ================================================================================================
struct AttnBwdDkvArgs {
    int S, h, S_pad;
    float scale_log2, scale;
    const float* stat_l2;      // [h][S_pad]
    const float* stat_delta;   // [h][S_pad]
    __nv_bfloat16* dkv;        // [S, h*256]: per head dK_nope (128) then dV (128)
    float* dk_rope;            // [h][S][64]
    unsigned int* status;
};

struct AttnBwdDkvSmem {
    static constexpr int kSlab128 = 128 * 128;                 // 128 rows x 128 B
    static constexpr int kSlab64 = 64 * 128;                   // 64 rows x 128 B
    static constexpr int kK = 0;                               // 3 slabs of 128 rows
    static constexpr int kV = kK + 3 * kSlab128;               // 2 slabs of 128 rows
    static constexpr int kQ = kV + 2 * kSlab128;               // 2 stages x 3 slabs of 64 rows
    static constexpr int kDO = kQ + 2 * 3 * kSlab64;           // 2 stages x 2 slabs of 64 rows
    static constexpr int kPt = kDO + 2 * 2 * kSlab64;          // P^T  [128 keys x 64 q]
    static constexpr int kDSt = kPt + kSlab128;                // dS^T [128 keys x 64 q]
    static constexpr int kStat = kDSt + kSlab128;              // 2 stages x (64 l2 + 64 delta) floats
    static constexpr int kBar = kStat + 2 * 512;
    static constexpr int kTotalBytes = kBar + 256 + 1024;
};

template <bool kCausal>
__global__ void __launch_bounds__(192, 1)
attn_bwd_dkv_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                          const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                          const AttnBwdDkvArgs args) {
    using L = AttnBwdDkvSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* kv_full = bars + 0;
    uint64_t* qdo_full = bars + 1;    // [2]
    uint64_t* qdo_empty = bars + 3;   // [2]
    uint64_t* st_full = bars + 5;     // [2]
    uint64_t* st_free = bars + 7;     // [2]
    uint64_t* dp_full = bars + 9;
    uint64_t* dp_free = bars + 10;
    uint64_t* pds_full = bars + 11;
    uint64_t* pds_free = bars + 12;
    uint64_t* acc_done = bars + 13;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_tile = blockIdx.x, head = blockIdx.y;
    const int t0 = k_tile * 128;
    const int n_q64 = (args.S + 63) / 64;
    const int j_begin = kCausal ? (t0 / 64) : 0;
    const int n_iter = n_q64 - j_begin;              // >= 1 because t0 < S

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&qdo_full[s], 1); mbar_init(&qdo_empty[s], 1);
            mbar_init(&st_full[s], 1); mbar_init(&st_free[s], 128);
        }
        mbar_init(dp_full, 1); mbar_init(dp_free, 128);
        mbar_init(pds_full, 128); mbar_init(pds_free, 1);
        mbar_init(acc_done, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_do);
        tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_st = tmem_base;            // 2 x 64 columns
    const uint32_t tmem_dp = tmem_base + 128;      // 64 columns
    const uint32_t tmem_dk = tmem_base + 192;      // 192 columns
    const uint32_t tmem_dv = tmem_base + 384;      // 128 columns

    if (warp == 0) {
        if (elect_one()) {
            mbar_arrive_expect_tx(kv_full, 5 * L::kSlab128);
            tma_load_2d(smem + L::kK, &tmap_kv, kv_full, head * 256, t0);
            tma_load_2d(smem + L::kK + L::kSlab128, &tmap_kv, kv_full, head * 256 + 64, t0);
            tma_load_2d(smem + L::kK + 2 * L::kSlab128, &tmap_kpe, kv_full, 0, t0);
            tma_load_2d(smem + L::kV, &tmap_kv, kv_full, head * 256 + 128, t0);
            tma_load_2d(smem + L::kV + L::kSlab128, &tmap_kv, kv_full, head * 256 + 192, t0);
            for (int j = 0; j < n_iter; ++j) {
                const int s = j & 1;
                if (!mbar_wait(&qdo_empty[s], ((j >> 1) & 1) ^ 1, abort_flag, args.status, 0x40)) break;
                const int q0 = (j_begin + j) * 64;
                mbar_arrive_expect_tx(&qdo_full[s], 5 * L::kSlab64 + 512);
                uint8_t* sq = smem + L::kQ + s * 3 * L::kSlab64;
                uint8_t* sdo = smem + L::kDO + s * 2 * L::kSlab64;
                for (int c = 0; c < 3; ++c)
                    tma_load_2d(sq + c * L::kSlab64, &tmap_q, &qdo_full[s], head * 192 + c * 64, q0);
                for (int c = 0; c < 2; ++c)
                    tma_load_2d(sdo + c * L::kSlab64, &tmap_do, &qdo_full[s], head * 128 + c * 64, q0);
                float* stat = reinterpret_cast<float*>(smem + L::kStat + s * 512);
                bulk_load_1d(stat, args.stat_l2 + static_cast<size_t>(head) * args.S_pad + q0, 256, &qdo_full[s]);
                bulk_load_1d(stat + 64, args.stat_delta + static_cast<size_t>(head) * args.S_pad + q0, 256,
                             &qdo_full[s]);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, 0, 0);    // S^T, dP^T: both K-major
            constexpr uint32_t idesc_dv = make_idesc_bf16(128, 128, 0, 1);   // dV: A = P^T K-major, B = dO MN-major
            constexpr uint32_t idesc_dk = make_idesc_bf16(128, 192, 0, 1);   // dK: A = dS^T,     B = Q  MN-major
            const uint32_t sk = smem_u32(smem + L::kK), sv = smem_u32(smem + L::kV);
            const uint32_t spt = smem_u32(smem + L::kPt), sdst = smem_u32(smem + L::kDSt);
            auto issue_acc = [&](int j) -> bool {   // dV += P^T dO_j, dK += dS^T Q_j
                if (!mbar_wait(pds_full, j & 1, abort_flag, args.status, 0x50)) return false;
                tc_fence_after_sync();
                const int s = j & 1;
                const uint32_t sq = smem_u32(smem + L::kQ + s * 3 * L::kSlab64);
                const uint32_t sdo = smem_u32(smem + L::kDO + s * 2 * L::kSlab64);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss(tmem_dv, desc_k_major(spt + kk * 32), desc_mn_major(sdo + kk * 2048, L::kSlab64), idesc_dv,
                           (j > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss(tmem_dk, desc_k_major(sdst + kk * 32), desc_mn_major(sq + kk * 2048, L::kSlab64), idesc_dk,
                           (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&qdo_empty[s]);
                mma_commit(pds_free);
                return true;
            };
            bool ok = mbar_wait(kv_full, 0, abort_flag, args.status, 0x51);
            for (int j = 0; j < n_iter && ok; ++j) {
                const int s = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                ok = mbar_wait(&qdo_full[s], ph, abort_flag, args.status, 0x52) &&
                     mbar_wait(&st_free[s], ph ^ 1, abort_flag, args.status, 0x53);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sq = smem_u32(smem + L::kQ + s * 3 * L::kSlab64);
                const uint32_t sdo = smem_u32(smem + L::kDO + s * 2 * L::kSlab64);
#pragma unroll
                for (int kk = 0; kk < 12; ++kk)
                    mma_ss(tmem_st + s * 64, desc_k_major(sk + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sq + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_st, kk > 0 ? 1u : 0u);
                mma_commit(&st_full[s]);
                ok = mbar_wait(dp_free, (j & 1) ^ 1, abort_flag, args.status, 0x54);
                if (!ok) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss(tmem_dp, desc_k_major(sv + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sdo + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_st, kk > 0 ? 1u : 0u);
                mma_commit(dp_full);
                if (j > 0) ok = issue_acc(j - 1);
            }
            if (ok) ok = issue_acc(n_iter - 1);
            if (ok) mma_commit(acc_done);
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;         // key row inside the tile == TMEM lane
        const int t_idx = t0 + row;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        bool ok = true;
        for (int j = 0; j < n_iter; ++j) {
            const int s = j & 1;
            const int q0 = (j_begin + j) * 64;
            ok = mbar_wait_warp(&st_full[s], (j >> 1) & 1, abort_flag, args.status, 0x60);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[64];
            tmem_ld_x32(tmem_st + lane_addr + s * 64, sv);
            tmem_ld_x32(tmem_st + lane_addr + s * 64 + 32, sv + 32);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(&st_free[s]);
            // stat tile was delivered with Q/dO on qdo_full[s], which the MMA warp waited for before
            // S^T could complete; this wait makes those bulk-copy writes visible to this thread too.
            ok = mbar_wait_warp(&qdo_full[s], (j >> 1) & 1, abort_flag, args.status, 0x61);
            if (!ok) break;
            const float* stat = reinterpret_cast<const float*>(smem + L::kStat + s * 512);
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
            if (j > 0) {
                ok = mbar_wait_warp(pds_free, (j - 1) & 1, abort_flag, args.status, 0x62);
                if (!ok) break;
            }
#pragma unroll
            for (int c16 = 0; c16 < 8; ++c16) {
                uint4 val;
                val.x = pack_bf16x2(p[c16 * 8 + 0], p[c16 * 8 + 1]);
                val.y = pack_bf16x2(p[c16 * 8 + 2], p[c16 * 8 + 3]);
                val.z = pack_bf16x2(p[c16 * 8 + 4], p[c16 * 8 + 5]);
                val.w = pack_bf16x2(p[c16 * 8 + 6], p[c16 * 8 + 7]);
                *reinterpret_cast<uint4*>(smem + L::kPt + swz128_offset(row, c16)) = val;
            }
            ok = mbar_wait_warp(dp_full, j & 1, abort_flag, args.status, 0x63);
            if (!ok) break;
            tc_fence_after_sync();
            tmem_ld_x32(tmem_dp + lane_addr, sv);
            tmem_ld_x32(tmem_dp + lane_addr + 32, sv + 32);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(dp_free);
#pragma unroll
            for (int c16 = 0; c16 < 8; ++c16) {
                const float4 d0 = *reinterpret_cast<const float4*>(stat + 64 + c16 * 8);
                const float4 d1 = *reinterpret_cast<const float4*>(stat + 64 + c16 * 8 + 4);
                const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                float ds[8];
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    ds[e] = p[c16 * 8 + e] * (__uint_as_float(sv[c16 * 8 + e]) - dl[e]);
                uint4 val;
                val.x = pack_bf16x2(ds[0], ds[1]);
                val.y = pack_bf16x2(ds[2], ds[3]);
                val.z = pack_bf16x2(ds[4], ds[5]);
                val.w = pack_bf16x2(ds[6], ds[7]);
                *reinterpret_cast<uint4*>(smem + L::kDSt + swz128_offset(row, c16)) = val;
            }
            fence_proxy_async_smem();
            mbar_arrive(pds_full);
        }
        if (ok) ok = mbar_wait_warp(acc_done, 0, abort_flag, args.status, 0x64);
        if (ok) {
            tc_fence_after_sync();
            const bool valid = t_idx < args.S;
            __nv_bfloat16* dkv_row = args.dkv + static_cast<size_t>(t_idx) * args.h * 256 + head * 256;
            float* dkr_row = args.dk_rope + (static_cast<size_t>(head) * args.S + t_idx) * 64;
#pragma unroll 1
            for (int c = 0; c < 10; ++c) {            // 6 chunks of dK (4 nope + 2 rope), 4 chunks of dV
                uint32_t r[32];
                __syncwarp();
                tmem_ld_x32(tmem_dk + lane_addr + c * 32, r);   // dV follows dK in TMEM
                tmem_ld_wait();
                if (!valid) continue;
                if (c == 4 || c == 5) {
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        float4 w = make_float4(__uint_as_float(r[v * 4]) * args.scale, __uint_as_float(r[v * 4 + 1]) * args.scale,
                                               __uint_as_float(r[v * 4 + 2]) * args.scale, __uint_as_float(r[v * 4 + 3]) * args.scale);
                        reinterpret_cast<float4*>(dkr_row + (c - 4) * 32)[v] = w;
                    }
                } else {
                    const float mul = c < 4 ? args.scale : 1.0f;
                    __nv_bfloat16* dst = dkv_row + (c < 4 ? c * 32 : 128 + (c - 6) * 32);
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]) * mul, __uint_as_float(r[v * 8 + 1]) * mul);
                        w.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]) * mul, __uint_as_float(r[v * 8 + 3]) * mul);
                        w.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]) * mul, __uint_as_float(r[v * 8 + 5]) * mul);
                        w.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]) * mul, __uint_as_float(r[v * 8 + 7]) * mul);
                        reinterpret_cast<uint4*>(dst)[v] = w;
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
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
    __nv_bfloat16* dq;           // [S, h, 192]
    unsigned int* status;
};

struct AttnBwdDqSmem {
    static constexpr int kSlab128 = 128 * 128;
    static constexpr int kSlab64 = 64 * 128;
    static constexpr int kQ = 0;                               // 3 slabs of 128 rows
    static constexpr int kDO = kQ + 3 * kSlab128;              // 2 slabs of 128 rows
    static constexpr int kK = kDO + 2 * kSlab128;              // 2 stages x 3 slabs of 64 rows
    static constexpr int kV = kK + 2 * 3 * kSlab64;            // 2 stages x 2 slabs of 64 rows
    static constexpr int kDS = kV + 2 * 2 * kSlab64;           // dS [128 q x 64 keys]
    static constexpr int kBar = kDS + kSlab128;
    static constexpr int kTotalBytes = kBar + 256 + 1024;
};

template <bool kCausal>
__global__ void __launch_bounds__(192, 1)
attn_bwd_dq_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                         const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                         const AttnBwdDqArgs args) {
    using L = AttnBwdDqSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* qdo_full = bars + 0;
    uint64_t* kv_full = bars + 1;     // [2]
    uint64_t* kv_empty = bars + 3;    // [2]
    uint64_t* sdp_full = bars + 5;    // [2]
    uint64_t* sdp_free = bars + 7;    // [2]
    uint64_t* ds_full = bars + 9;
    uint64_t* ds_free = bars + 10;
    uint64_t* acc_done = bars + 11;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_q_tiles = (args.S + 127) / 128;
    const int q_tile = n_q_tiles - 1 - static_cast<int>(blockIdx.x);
    const int head = blockIdx.y;
    const int q0 = q_tile * 128;
    const int k_end = kCausal ? min(args.S, q0 + 128) : args.S;
    const int n_iter = (k_end + 63) / 64;

    if (threadIdx.x == 0) {
        mbar_init(qdo_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1);
            mbar_init(&sdp_full[s], 1); mbar_init(&sdp_free[s], 128);
        }
        mbar_init(ds_full, 128); mbar_init(ds_free, 1);
        mbar_init(acc_done, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_do);
        tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_s = tmem_base;             // 2 x 64 columns
    const uint32_t tmem_dp = tmem_base + 128;      // 2 x 64 columns
    const uint32_t tmem_dq = tmem_base + 256;      // 192 columns

    if (warp == 0) {
        if (elect_one()) {
            mbar_arrive_expect_tx(qdo_full, 5 * L::kSlab128);
            for (int c = 0; c < 3; ++c)
                tma_load_2d(smem + L::kQ + c * L::kSlab128, &tmap_q, qdo_full, head * 192 + c * 64, q0);
            for (int c = 0; c < 2; ++c)
                tma_load_2d(smem + L::kDO + c * L::kSlab128, &tmap_do, qdo_full, head * 128 + c * 64, q0);
            for (int j = 0; j < n_iter; ++j) {
                const int s = j & 1;
                if (!mbar_wait(&kv_empty[s], ((j >> 1) & 1) ^ 1, abort_flag, args.status, 0x70)) break;
                mbar_arrive_expect_tx(&kv_full[s], 5 * L::kSlab64);
                uint8_t* sk = smem + L::kK + s * 3 * L::kSlab64;
                uint8_t* sv = smem + L::kV + s * 2 * L::kSlab64;
                tma_load_2d(sk, &tmap_kv, &kv_full[s], head * 256, j * 64);
                tma_load_2d(sk + L::kSlab64, &tmap_kv, &kv_full[s], head * 256 + 64, j * 64);
                tma_load_2d(sk + 2 * L::kSlab64, &tmap_kpe, &kv_full[s], 0, j * 64);
                tma_load_2d(sv, &tmap_kv, &kv_full[s], head * 256 + 128, j * 64);
                tma_load_2d(sv + L::kSlab64, &tmap_kv, &kv_full[s], head * 256 + 192, j * 64);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 64, 0, 0);     // S, dP: both K-major
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 192, 0, 1);   // dQ: A = dS K-major, B = K MN-major
            const uint32_t sq = smem_u32(smem + L::kQ), sdo = smem_u32(smem + L::kDO);
            const uint32_t sds = smem_u32(smem + L::kDS);
            auto issue_dq = [&](int j) -> bool {
                if (!mbar_wait(ds_full, j & 1, abort_flag, args.status, 0x80)) return false;
                tc_fence_after_sync();
                const int s = j & 1;
                const uint32_t sk = smem_u32(smem + L::kK + s * 3 * L::kSlab64);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss(tmem_dq, desc_k_major(sds + kk * 32), desc_mn_major(sk + kk * 2048, L::kSlab64), idesc_dq,
                           (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&kv_empty[s]);
                mma_commit(ds_free);
                return true;
            };
            bool ok = mbar_wait(qdo_full, 0, abort_flag, args.status, 0x81);
            for (int j = 0; j < n_iter && ok; ++j) {
                const int s = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                ok = mbar_wait(&kv_full[s], ph, abort_flag, args.status, 0x82) &&
                     mbar_wait(&sdp_free[s], ph ^ 1, abort_flag, args.status, 0x83);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sk = smem_u32(smem + L::kK + s * 3 * L::kSlab64);
                const uint32_t sv = smem_u32(smem + L::kV + s * 2 * L::kSlab64);
#pragma unroll
                for (int kk = 0; kk < 12; ++kk)
                    mma_ss(tmem_s + s * 64, desc_k_major(sq + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sk + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_s, kk > 0 ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss(tmem_dp + s * 64, desc_k_major(sdo + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sv + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_s, kk > 0 ? 1u : 0u);
                mma_commit(&sdp_full[s]);
                if (j > 0) ok = issue_dq(j - 1);
            }
            if (ok) ok = issue_dq(n_iter - 1);
            if (ok) mma_commit(acc_done);
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int s_idx = q0 + row;
        const bool valid = s_idx < args.S;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        // Rows past the end of the sequence get LSE = +inf so that their P is exactly zero.
        const float l2 = valid ? args.lse[static_cast<size_t>(s_idx) * args.h + head] * 1.4426950408889634f : INFINITY;
        const float delta = valid ? args.stat_delta[static_cast<size_t>(head) * args.S_pad + s_idx] : 0.f;
        bool ok = true;
        for (int j = 0; j < n_iter; ++j) {
            const int s = j & 1;
            ok = mbar_wait_warp(&sdp_full[s], (j >> 1) & 1, abort_flag, args.status, 0x90);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[64], dpv[64];
            tmem_ld_x32(tmem_s + lane_addr + s * 64, sv);
            tmem_ld_x32(tmem_s + lane_addr + s * 64 + 32, sv + 32);
            tmem_ld_x32(tmem_dp + lane_addr + s * 64, dpv);
            tmem_ld_x32(tmem_dp + lane_addr + s * 64 + 32, dpv + 32);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(&sdp_free[s]);
            const int tk0 = j * 64;
            const bool edge = (kCausal && tk0 + 63 > q0) || (tk0 + 64 > args.S);
            uint32_t pk[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                float d[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int cc = 2 * c + e;
                    float p = fast_exp2(fmaf(__uint_as_float(sv[cc]), args.scale_log2, -l2));
                    if (edge) {
                        const int t = tk0 + cc;
                        if ((kCausal && t > s_idx) || t >= args.S) p = 0.f;
                    }
                    d[e] = p * (__uint_as_float(dpv[cc]) - delta);
                }
                pk[c] = pack_bf16x2(d[0], d[1]);
            }
            if (j > 0) {
                ok = mbar_wait_warp(ds_free, (j - 1) & 1, abort_flag, args.status, 0x91);
                if (!ok) break;
            }
#pragma unroll
            for (int c16 = 0; c16 < 8; ++c16) {
                uint4 val = make_uint4(pk[c16 * 4], pk[c16 * 4 + 1], pk[c16 * 4 + 2], pk[c16 * 4 + 3]);
                *reinterpret_cast<uint4*>(smem + L::kDS + swz128_offset(row, c16)) = val;
            }
            fence_proxy_async_smem();
            mbar_arrive(ds_full);
        }
        if (ok) ok = mbar_wait_warp(acc_done, 0, abort_flag, args.status, 0x92);
        if (ok) {
            tc_fence_after_sync();
            __nv_bfloat16* dst = args.dq + (static_cast<size_t>(s_idx) * args.h + head) * 192;
#pragma unroll 1
            for (int c = 0; c < 6; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_x32(tmem_dq + lane_addr + c * 32, r);
                tmem_ld_wait();
                if (!valid) continue;
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]) * args.scale, __uint_as_float(r[v * 8 + 1]) * args.scale);
                    w.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]) * args.scale, __uint_as_float(r[v * 8 + 3]) * args.scale);
                    w.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]) * args.scale, __uint_as_float(r[v * 8 + 5]) * args.scale);
                    w.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]) * args.scale, __uint_as_float(r[v * 8 + 7]) * args.scale);
                    reinterpret_cast<uint4*>(dst + c * 32)[v] = w;
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace laga
