// Backward of Algorithm 1 step 5 (Section 5.2: the chain rule through the softmax attention) for
// the DeepSeek-V3 head geometry, as two tcgen05 kernels that recompute P from the saved LSE:
//
//   attn_bwd_dkv  one CTA per (128-key tile, head), sweeping the 64-row query tiles that attend to it:
//                 S^T = K Q^T, dP^T = V dO^T, P^T = exp(scale S^T - LSE), dS^T = P^T (dP^T - delta),
//                 dV += P^T dO, dK += dS^T Q  (dK 192 wide: 128 nope columns + 64 rope columns).
//                 TMEM lanes are keys, so LSE and delta are per-column vectors staged in shared memory.
//   attn_bwd_dq   one CTA per (128-query tile, head), sweeping 128-key tiles:
//                 S = Q K^T, dP = dO V^T, dS = P (dP - delta), dQ += dS K.  TMEM lanes are queries.
//
// Both read K_nope / V from the recomputed bf16 up-projection KV[S, h*256] and the shared rope band
// from k_pe[S, 64]; both keep every accumulator in TMEM and never materialise S x S.
//
// Roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 and 6..9 two consumer
// warpgroups (every thread owns one TMEM lane).  P^T / dS^T (dkv) and dS (dq) never touch shared
// memory: the consumers write them back to TMEM as packed bf16 and the accumulating MMAs read their
// A operand from there.  Scratch columns are reused by an MMA that the same thread issues after the
// MMAs that read them; the tensor pipe runs one thread's MMAs in order, so that reuse needs no barrier.
//   dkv: dK (192) + dV (128) leave 192 TMEM columns, so query tiles are 64 rows and the two groups
//        take alternate tiles (scratch 2 x 64 columns + P^T 2 x 32): one group's exponentials overlap
//        the other's MMAs.  A 64-wide N costs 48 cycles per MMA against 32 ideal.
//   dq:  128-key tiles, all MMAs 128 wide; the two groups take 64 key columns each.  dO (the A
//        operand of dP) lives in TMEM, which frees shared memory for a third K stage.
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
// Eight lanes per (row, head): each lane reads 16 channels of O and dO as two 16-byte loads apiece.
__global__ void __launch_bounds__(256)
bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                 const float* __restrict__ lse, int S, int h, int S_pad, float* __restrict__ stat_l2,
                 float* __restrict__ stat_delta) {
    const long long item = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 3;   // (row, head) pair
    const int sub = threadIdx.x & 7;
    const bool live = item < static_cast<long long>(S_pad) * h;
    const int s = live ? static_cast<int>(item / h) : 0, i = live ? static_cast<int>(item % h) : 0;
    float acc = 0.f;
    if (live && s < S) {
        const size_t base = (static_cast<size_t>(s) * h + i) * 128 + sub * 16;
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
        const bool valid = s < S;
        stat_l2[static_cast<size_t>(i) * S_pad + s] = valid ? lse[static_cast<size_t>(s) * h + i] * 1.4426950408889634f : INFINITY;
        stat_delta[static_cast<size_t>(i) * S_pad + s] = valid ? acc : 0.f;
    }
}

// dk_pe[t, r] is the sum over heads of the rope-column key gradients (Section 5.3: the rope band is
// shared by every head, so its gradient is the sum over the head shard).  The dK/dV kernel adds each
// head's columns into an fp32 accumulator with atomics; this kernel rounds the sums to bf16.
__global__ void __launch_bounds__(256)
bwd_dkpe_convert_kernel(const float* __restrict__ dkpe_acc, int S, __nv_bfloat16* __restrict__ dk_pe) {
    const size_t idx = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
    if (idx >= static_cast<size_t>(S) * 64) return;
    const float4 v = *reinterpret_cast<const float4*>(dkpe_acc + idx);
    uint2 o;
    o.x = pack_bf16x2(v.x, v.y);
    o.y = pack_bf16x2(v.z, v.w);
    *reinterpret_cast<uint2*>(dk_pe + idx) = o;
}

// Deterministic alternative to the atomics: sum the per-head buffers in head order.
__global__ void __launch_bounds__(256)
bwd_dkpe_reduce_kernel(const float* __restrict__ dk_rope, int S, int h, __nv_bfloat16* __restrict__ dk_pe) {
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t n = static_cast<size_t>(S) * 64;
    if (idx >= n) return;
    float acc = 0.f;
    for (int i = 0; i < h; ++i) acc += dk_rope[static_cast<size_t>(i) * n + idx];
    dk_pe[idx] = __float2bfloat16_rn(acc);
}

constexpr int kBwdThreads = 320;
constexpr int kBwdStages = 3;

// ================================================================================================
// dK / dV kernel
// ================================================================================================
struct AttnBwdDkvArgs {
    int S, h, S_pad;
    float scale_log2, scale;
    const float* stat_l2;      // [h][S_pad]
    const float* stat_delta;   // [h][S_pad]
    __nv_bfloat16* dkv;        // [S, h*256]: per head dK_nope (128) then dV (128)
    float* dkpe_acc;           // [S][64] fp32, zeroed by the host; every head's CTA adds into it
    float* dk_rope_per_head;   // deterministic mode: [h][S][64] fp32 written per head (then summed in a fixed
                               // order by bwd_dkpe_reduce_kernel); nullptr selects the atomic path
    unsigned int* status;
};

struct AttnBwdDkvSmem {
    static constexpr int kSlab128 = 128 * 128;                 // 128 rows x 128 B
    static constexpr int kSlab64 = 64 * 128;                   // 64 rows x 128 B
    static constexpr int kStage = 5 * kSlab64;                 // Q (3 slabs) + dO (2 slabs), 64 rows each
    static constexpr int kK = 0;                               // 3 slabs of 128 rows
    static constexpr int kV = kK + 3 * kSlab128;               // 2 slabs of 128 rows
    static constexpr int kQdO = kV + 2 * kSlab128;             // kBwdStages stages
    static constexpr int kStat = kQdO + kBwdStages * kStage;   // per stage: 64 l2 + 64 delta floats
    static constexpr int kBar = kStat + kBwdStages * 512;
    static constexpr int kTotalBytes = kBar + 256 + 1024;
};

template <bool kCausal>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_dkv_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                          const __grid_constant__ CUtensorMap tmap_kv, const __grid_constant__ CUtensorMap tmap_kpe,
                          const AttnBwdDkvArgs args) {
    using L = AttnBwdDkvSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* kv_full = bars + 0;
    uint64_t* qdo_full = bars + 1;    // [3]
    uint64_t* qdo_empty = bars + 4;   // [3]
    uint64_t* st_full = bars + 7;     // [2]  S^T of the group's tile is in TMEM
    uint64_t* st_read = bars + 9;     // [2]  the group has loaded it: the columns may take dP^T
    uint64_t* p_full = bars + 11;     // [2]  P^T (bf16) is in TMEM
    uint64_t* dp_full = bars + 13;    // [2]  dP^T is in TMEM
    uint64_t* ds_full = bars + 15;    // [2]  dS^T (bf16) is in TMEM
    uint64_t* acc_done = bars + 17;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_tile = blockIdx.x, head = blockIdx.y;
    const int t0 = k_tile * 128;
    const int n_q64 = (args.S + 63) / 64;
    const int j_begin = kCausal ? (t0 / 64) : 0;
    const int n_iter = n_q64 - j_begin;              // >= 1 because t0 < S

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < kBwdStages; ++s) { mbar_init(&qdo_full[s], 1); mbar_init(&qdo_empty[s], 1); }
        for (int g = 0; g < 2; ++g) {
            mbar_init(&st_full[g], 1); mbar_init(&st_read[g], 128); mbar_init(&p_full[g], 128);
            mbar_init(&dp_full[g], 1); mbar_init(&ds_full[g], 128);
        }
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
    // columns: [0,64) group 0 scratch (S^T, then dP^T, then dS^T bf16) | [64,128) group 1 scratch |
    //          [128,160) P^T group 0 | [160,192) P^T group 1 | [192,384) dK | [384,512) dV
    const uint32_t tmem_pt = tmem_base + 128;
    const uint32_t tmem_dk = tmem_base + 192;
    const uint32_t tmem_dv = tmem_base + 384;

    if (warp == 0) {
        if (elect_one()) {
            mbar_arrive_expect_tx(kv_full, 5 * L::kSlab128);
            tma_load_2d(smem + L::kK, &tmap_kv, kv_full, head * 256, t0);
            tma_load_2d(smem + L::kK + L::kSlab128, &tmap_kv, kv_full, head * 256 + 64, t0);
            tma_load_2d(smem + L::kK + 2 * L::kSlab128, &tmap_kpe, kv_full, 0, t0);
            tma_load_2d(smem + L::kV, &tmap_kv, kv_full, head * 256 + 128, t0);
            tma_load_2d(smem + L::kV + L::kSlab128, &tmap_kv, kv_full, head * 256 + 192, t0);
            for (int j = 0; j < n_iter; ++j) {
                const int st = j % kBwdStages;
                if (!mbar_wait(&qdo_empty[st], ((j / kBwdStages) & 1) ^ 1, abort_flag, args.status, 0x40)) break;
                const int q0 = (j_begin + j) * 64;
                mbar_arrive_expect_tx(&qdo_full[st], L::kStage + 512);
                uint8_t* sq = smem + L::kQdO + st * L::kStage;
                uint8_t* sdo = sq + 3 * L::kSlab64;
                for (int c = 0; c < 3; ++c)
                    tma_load_2d(sq + c * L::kSlab64, &tmap_q, &qdo_full[st], head * 192 + c * 64, q0);
                for (int c = 0; c < 2; ++c)
                    tma_load_2d(sdo + c * L::kSlab64, &tmap_do, &qdo_full[st], head * 128 + c * 64, q0);
                float* stat = reinterpret_cast<float*>(smem + L::kStat + st * 512);
                bulk_load_1d(stat, args.stat_l2 + static_cast<size_t>(head) * args.S_pad + q0, 256, &qdo_full[st]);
                bulk_load_1d(stat + 64, args.stat_delta + static_cast<size_t>(head) * args.S_pad + q0, 256,
                             &qdo_full[st]);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_st = make_idesc_bf16(128, 64, 0, 0);    // S^T, dP^T: both K-major
            constexpr uint32_t idesc_dv = make_idesc_bf16(128, 128, 0, 1);   // dV: A = P^T (TMEM), B = dO MN-major
            constexpr uint32_t idesc_dk = make_idesc_bf16(128, 192, 0, 1);   // dK: A = dS^T (TMEM), B = Q MN-major
            const uint32_t sk = smem_u32(smem + L::kK), sv = smem_u32(smem + L::kV);
            auto stage_q = [&](int j) { return smem_u32(smem + L::kQdO + (j % kBwdStages) * L::kStage); };
            auto issue_st = [&](int j) -> bool {     // S^T(j) = K Q_j^T into the group's scratch columns
                const int g = j & 1;
                if (!mbar_wait(&qdo_full[j % kBwdStages], (j / kBwdStages) & 1, abort_flag, args.status, 0x52))
                    return false;
                tc_fence_after_sync();
                const uint32_t sq = stage_q(j);
#pragma unroll
                for (int kk = 0; kk < 12; ++kk)
                    mma_ss(tmem_base + g * 64, desc_k_major(sk + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sq + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_st, kk > 0 ? 1u : 0u);
                mma_commit(&st_full[g]);
                return true;
            };
            auto issue_dp = [&](int j) -> bool {     // dP^T(j) = V dO_j^T over the same columns once S^T was read
                const int g = j & 1;
                if (!mbar_wait(&st_read[g], (j >> 1) & 1, abort_flag, args.status, 0x53)) return false;
                tc_fence_after_sync();
                const uint32_t sdo = stage_q(j) + 3 * L::kSlab64;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss(tmem_base + g * 64, desc_k_major(sv + (kk >> 2) * L::kSlab128 + (kk & 3) * 32),
                           desc_k_major(sdo + (kk >> 2) * L::kSlab64 + (kk & 3) * 32), idesc_st, kk > 0 ? 1u : 0u);
                mma_commit(&dp_full[g]);
                return true;
            };
            auto issue_dv = [&](int j) -> bool {     // dV += P^T dO_j (A operand from TMEM)
                const int g = j & 1;
                if (!mbar_wait(&p_full[g], (j >> 1) & 1, abort_flag, args.status, 0x50)) return false;
                tc_fence_after_sync();
                const uint32_t sdo = stage_q(j) + 3 * L::kSlab64;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts(tmem_dv, tmem_pt + g * 32 + kk * 8, desc_mn_major(sdo + kk * 2048, L::kSlab64), idesc_dv,
                           (j > 0 || kk > 0) ? 1u : 0u);
                return true;
            };
            auto issue_dk = [&](int j) -> bool {     // dK += dS^T Q_j (A operand from TMEM)
                const int g = j & 1;
                if (!mbar_wait(&ds_full[g], (j >> 1) & 1, abort_flag, args.status, 0x51)) return false;
                tc_fence_after_sync();
                const uint32_t sq = stage_q(j);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts(tmem_dk, tmem_base + g * 64 + kk * 8, desc_mn_major(sq + kk * 2048, L::kSlab64), idesc_dk,
                           (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&qdo_empty[j % kBwdStages]);
                return true;
            };
            // Issue order per tile: S^T(j), dV(j-1), dP^T(j), dK(j-1).  dV(j-1) gives this tile's warpgroup
            // time to load S^T(j) before dP^T(j) overwrites it, and dK(j-1) comes last so that the other
            // warpgroup has S^T(j), dV(j-1) and dP^T(j) -- some 1200 clocks -- to turn dP^T(j-1) into dS^T(j-1).
            bool ok = mbar_wait(kv_full, 0, abort_flag, args.status, 0x54);
            for (int j = 0; j < n_iter && ok; ++j) {
                ok = issue_st(j);
                if (ok && j > 0) ok = issue_dv(j - 1);
                if (ok) ok = issue_dp(j);
                if (ok && j > 0) ok = issue_dk(j - 1);
            }
            if (ok) ok = issue_dv(n_iter - 1);
            if (ok) ok = issue_dk(n_iter - 1);
            if (ok) mma_commit(acc_done);
        }
    } else {
        const int g = (warp - 2) >> 2;               // consumer warpgroup 0 or 1
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;         // key row inside the tile == TMEM lane
        const int t_idx = t0 + row;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        const uint32_t tmem_scr = tmem_base + g * 64 + lane_addr;
        bool ok = true;
        for (int j = g; j < n_iter; j += 2) {
            const uint32_t ph = (j >> 1) & 1;
            const int st = j % kBwdStages;
            const int q0 = (j_begin + j) * 64;
            ok = mbar_wait_warp(&st_full[g], ph, abort_flag, args.status, 0x60);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[64];
            tmem_ld_x32(tmem_scr, sv);
            tmem_ld_x32(tmem_scr + 32, sv + 32);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(&st_read[g]);
            // The statistics arrived with Q/dO on qdo_full[st]; waiting on it here makes those
            // bulk-copy writes visible to this thread as well.
            ok = mbar_wait_warp(&qdo_full[st], (j / kBwdStages) & 1, abort_flag, args.status, 0x61);
            if (!ok) break;
            const float* stat = reinterpret_cast<const float*>(smem + L::kStat + st * 512);
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
            tmem_st_x32(tmem_pt + g * 32 + lane_addr, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&p_full[g]);

            ok = mbar_wait_warp(&dp_full[g], ph, abort_flag, args.status, 0x63);
            if (!ok) break;
            tc_fence_after_sync();
            tmem_ld_x32(tmem_scr, sv);
            tmem_ld_x32(tmem_scr + 32, sv + 32);
            tmem_ld_wait();
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                const float4 d0 = *reinterpret_cast<const float4*>(stat + 64 + c8 * 8);
                const float4 d1 = *reinterpret_cast<const float4*>(stat + 64 + c8 * 8 + 4);
                const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int c = c8 * 8 + 2 * e;
                    pk[c8 * 4 + e] = pack_bf16x2(p[c] * (__uint_as_float(sv[c]) - dl[2 * e]),
                                                 p[c + 1] * (__uint_as_float(sv[c + 1]) - dl[2 * e + 1]));
                }
            }
            tmem_st_x32(tmem_scr, pk);               // dS^T over the first 32 of the columns dP^T occupied
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&ds_full[g]);
        }
        if (ok) ok = mbar_wait_warp(acc_done, 0, abort_flag, args.status, 0x64);
        if (ok) {
            tc_fence_after_sync();
            const bool valid = t_idx < args.S;
            __nv_bfloat16* dkv_row = args.dkv + static_cast<size_t>(t_idx) * args.h * 256 + head * 256;
            float* dkr_row = args.dkpe_acc + static_cast<size_t>(t_idx) * 64;
            // 10 chunks of 32 columns: dK nope (0..3), dK rope (4..5), dV (6..9; dV follows dK in TMEM).
            // Group 0 drains chunks 0..4, group 1 chunks 5..9.
#pragma unroll 1
            for (int c = g * 5; c < g * 5 + 5; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_x32(tmem_dk + lane_addr + c * 32, r);
                tmem_ld_wait();
                if (!valid) continue;
                if (c == 4 || c == 5) {
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        float4 w = make_float4(__uint_as_float(r[v * 4]) * args.scale, __uint_as_float(r[v * 4 + 1]) * args.scale,
                                               __uint_as_float(r[v * 4 + 2]) * args.scale, __uint_as_float(r[v * 4 + 3]) * args.scale);
                        if (args.dk_rope_per_head != nullptr)
                            reinterpret_cast<float4*>(args.dk_rope_per_head +
                                                      (static_cast<size_t>(head) * args.S + t_idx) * 64 + (c - 4) * 32)[v] = w;
                        else
                            atomicAdd(reinterpret_cast<float4*>(dkr_row + (c - 4) * 32) + v, w);
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
    const __nv_bfloat16* dout;   // [S, h, 128]
    __nv_bfloat16* dq;           // [S, h, 192]
    unsigned int* status;
};

constexpr int kDqKStages = 3;

struct AttnBwdDqSmem {
    static constexpr int kSlab = 128 * 128;
    static constexpr int kQ = 0;                               // 3 slabs
    static constexpr int kK = kQ + 3 * kSlab;                  // 3 stages x 3 slabs
    static constexpr int kV = kK + kDqKStages * 3 * kSlab;     // 1 stage x 2 slabs
    static constexpr int kBar = kV + 2 * kSlab;
    static constexpr int kTotalBytes = kBar + 256 + 1024;
};

// dO of the query tile is the A operand of dP = dO V^T for every key tile.  It is kept in TMEM as
// packed bf16 (64 columns) instead of 32 KB of shared memory, which is what leaves room for a third
// stage of K: a K tile lives from its score MMA to its dQ MMA, a whole tile period later.
template <bool kCausal>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_dq_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                         const __grid_constant__ CUtensorMap tmap_kpe, const AttnBwdDqArgs args) {
    using L = AttnBwdDqSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBar);
    uint64_t* q_full = bars + 0;
    uint64_t* k_full = bars + 1;      // [3]
    uint64_t* k_empty = bars + 4;     // [3]
    uint64_t* v_full = bars + 7;
    uint64_t* v_empty = bars + 8;
    uint64_t* do_ready = bars + 9;    // dO is in TMEM
    uint64_t* s_full = bars + 10;     // S is in TMEM
    uint64_t* s_read = bars + 11;     // both groups have loaded it
    uint64_t* dp_full = bars + 12;    // dP is in TMEM
    uint64_t* ds_full = bars + 13;    // dS (bf16) is in TMEM
    uint64_t* acc_done = bars + 14;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_q_tiles = (args.S + 127) / 128;
    const int q_tile = n_q_tiles - 1 - static_cast<int>(blockIdx.x);
    const int head = blockIdx.y;
    const int q0 = q_tile * 128;
    const int n_iter = kCausal ? q_tile + 1 : n_q_tiles;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kDqKStages; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
        mbar_init(v_full, 1); mbar_init(v_empty, 1);
        mbar_init(do_ready, 256);
        mbar_init(s_full, 1); mbar_init(s_read, 256); mbar_init(dp_full, 1); mbar_init(ds_full, 256);
        mbar_init(acc_done, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_kv); tma_prefetch_desc(&tmap_kpe);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // columns: [0,128) S | [128,256) dP, then dS as bf16 (keys 0..63 in [128,160), 64..127 in [192,224)) |
    //          [256,320) dO as bf16 | [320,512) dQ
    const uint32_t tmem_dp = tmem_base + 128;
    const uint32_t tmem_do = tmem_base + 256;
    const uint32_t tmem_dq = tmem_base + 320;

    if (warp == 0) {
        if (elect_one()) {
            mbar_arrive_expect_tx(q_full, 3 * L::kSlab);
            for (int c = 0; c < 3; ++c)
                tma_load_2d(smem + L::kQ + c * L::kSlab, &tmap_q, q_full, head * 192 + c * 64, q0);
            auto load_k = [&](int j) -> bool {
                const int st = j % kDqKStages;
                if (!mbar_wait(&k_empty[st], ((j / kDqKStages) & 1) ^ 1, abort_flag, args.status, 0x70)) return false;
                mbar_arrive_expect_tx(&k_full[st], 3 * L::kSlab);
                uint8_t* sk = smem + L::kK + st * 3 * L::kSlab;
                tma_load_2d(sk, &tmap_kv, &k_full[st], head * 256, j * 128);
                tma_load_2d(sk + L::kSlab, &tmap_kv, &k_full[st], head * 256 + 64, j * 128);
                tma_load_2d(sk + 2 * L::kSlab, &tmap_kpe, &k_full[st], 0, j * 128);
                return true;
            };
            bool ok = load_k(0);
            for (int j = 0; j < n_iter && ok; ++j) {
                if (j + 1 < n_iter) ok = load_k(j + 1);
                if (!ok) break;
                ok = mbar_wait(v_empty, (j & 1) ^ 1, abort_flag, args.status, 0x71);
                if (!ok) break;
                mbar_arrive_expect_tx(v_full, 2 * L::kSlab);
                tma_load_2d(smem + L::kV, &tmap_kv, v_full, head * 256 + 128, j * 128);
                tma_load_2d(smem + L::kV + L::kSlab, &tmap_kv, v_full, head * 256 + 192, j * 128);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);    // S: both K-major; dP: A from TMEM
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, 192, 0, 1);   // dQ: A = dS (TMEM), B = K MN-major
            const uint32_t sq = smem_u32(smem + L::kQ);
            const uint32_t sv = smem_u32(smem + L::kV);
            auto stage_k = [&](int j) { return smem_u32(smem + L::kK + (j % kDqKStages) * 3 * L::kSlab); };
            auto issue_s = [&](int j) -> bool {      // S(j) = Q K_j^T
                if (!mbar_wait(&k_full[j % kDqKStages], (j / kDqKStages) & 1, abort_flag, args.status, 0x82)) return false;
                if (j > 0 && !mbar_wait(s_read, (j - 1) & 1, abort_flag, args.status, 0x83)) return false;
                tc_fence_after_sync();
                const uint32_t sk = stage_k(j);
#pragma unroll
                for (int kk = 0; kk < 12; ++kk) {
                    const uint32_t off = (kk >> 2) * L::kSlab + (kk & 3) * 32;
                    mma_ss(tmem_base, desc_k_major(sq + off), desc_k_major(sk + off), idesc_s, kk > 0 ? 1u : 0u);
                }
                mma_commit(s_full);
                return true;
            };
            auto issue_dp = [&](int j) -> bool {     // dP(j) = dO V_j^T; overwrites dS(j-1), whose reader was issued earlier
                if (!mbar_wait(v_full, j & 1, abort_flag, args.status, 0x84)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem_dp, tmem_do + kk * 8, desc_k_major(sv + (kk >> 2) * L::kSlab + (kk & 3) * 32), idesc_s,
                           kk > 0 ? 1u : 0u);
                mma_commit(v_empty);
                mma_commit(dp_full);
                return true;
            };
            bool ok = mbar_wait(q_full, 0, abort_flag, args.status, 0x81) &&
                      mbar_wait(do_ready, 0, abort_flag, args.status, 0x85);
            if (ok) ok = issue_s(0);
            if (ok) ok = issue_dp(0);
            for (int j = 0; j < n_iter && ok; ++j) {
                if (j + 1 < n_iter) ok = issue_s(j + 1);
                if (!ok) break;
                ok = mbar_wait(ds_full, j & 1, abort_flag, args.status, 0x80);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sk = stage_k(j);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem_dq, tmem_dp + (kk >> 2) * 64 + (kk & 3) * 8, desc_mn_major(sk + kk * 2048, L::kSlab),
                           idesc_dq, (j > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&k_empty[j % kDqKStages]);
                if (j + 1 < n_iter) ok = issue_dp(j + 1);
            }
            if (ok) mma_commit(acc_done);
        }
    } else {
        const int g = (warp - 2) >> 2;               // consumer group: key columns [64g, 64g+64) of the tile
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int s_idx = q0 + row;
        const bool valid = s_idx < args.S;
        const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
        {   // this thread's dO row, channels [64g, 64g+64), as 32 packed words into TMEM
            uint32_t w[32];
            if (valid) {
                const uint4* src = reinterpret_cast<const uint4*>(args.dout + (static_cast<size_t>(s_idx) * args.h + head) * 128 + g * 64);
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
            tmem_st_x32(tmem_do + lane_addr + g * 32, w);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(do_ready);
        }
        // Rows past the end of the sequence get LSE = +inf so that their P is exactly zero.
        const float l2 = valid ? args.lse[static_cast<size_t>(s_idx) * args.h + head] * 1.4426950408889634f : INFINITY;
        const float delta = valid ? args.stat_delta[static_cast<size_t>(head) * args.S_pad + s_idx] : 0.f;
        bool ok = true;
        for (int j = 0; j < n_iter; ++j) {
            ok = mbar_wait_warp(s_full, j & 1, abort_flag, args.status, 0x90);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[64];
            tmem_ld_x32(tmem_base + lane_addr + g * 64, sv);
            tmem_ld_x32(tmem_base + lane_addr + g * 64 + 32, sv + 32);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(s_read);
            const int tk0 = j * 128 + g * 64;
            const bool edge = (kCausal && tk0 + 63 > q0) || (tk0 + 64 > args.S);
            float p[64];
#pragma unroll
            for (int c = 0; c < 64; ++c) {
                float v = fast_exp2(fmaf(__uint_as_float(sv[c]), args.scale_log2, -l2));
                if (edge) {
                    const int t = tk0 + c;
                    if ((kCausal && t > s_idx) || t >= args.S) v = 0.f;
                }
                p[c] = v;
            }
            ok = mbar_wait_warp(dp_full, j & 1, abort_flag, args.status, 0x91);
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
        if (ok) ok = mbar_wait_warp(acc_done, 0, abort_flag, args.status, 0x92);
        if (ok) {
            tc_fence_after_sync();
            __nv_bfloat16* dst = args.dq + (static_cast<size_t>(s_idx) * args.h + head) * 192;
#pragma unroll 1
            for (int c = g * 3; c < g * 3 + 3; ++c) {   // six 32-column chunks, three per group
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
