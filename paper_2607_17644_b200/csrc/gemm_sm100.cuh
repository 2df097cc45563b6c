// Dense bf16 x bf16 -> fp32 GEMM on tcgen05 tensor cores with TMEM accumulators, fed by TMA.
// Used for the three contractions with the latent (Algorithm 1 step 4 and its two transposes in
// the backward of Section 5.2):
//     KV    [S, N]   = c_kv [S, d_c] . W [d_c, N]          A K-major,  B MN-major, bf16 out
//     dc_kv [S, d_c] = dKV  [S, N]   . W^T                 A K-major,  B K-major,  bf16 out
//     dW    [d_c, N] = c_kv^T . dKV                        A MN-major, B MN-major, fp32 atomic out (split-K)
//
// One CTA computes one 128 x BN output tile over a K range.  Warp 0 issues TMA loads, warp 1 issues
// the MMAs, warps 2..5 drain the accumulator from TMEM (each warp owns the 32 TMEM lanes its
// warp-id-mod-4 selects).  Operand tiles are 64 K-elements deep, 128-byte swizzled, STAGES deep.
#pragma once
#include "sm100_ptx.cuh"

namespace laga {

struct GemmArgs {
    int M, N, K;          // problem size; M may be ragged, N % BN == 0, K tail is zero-filled by TMA
    int k_tiles_per_split;
    void* C;              // bf16 [M, ldc] (EPI_BF16) or fp32 [M, ldc] (EPI_ATOMIC_F32)
    int ldc;
    unsigned int* status;
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
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::kBarrierOffset);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_bar = empty_bar + STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_bar + 1);
    AbortFlag* abort_flag = reinterpret_cast<AbortFlag*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * 128;
    const int total_k_tiles = (args.K + 63) / 64;
    const int kt_begin = blockIdx.z * args.k_tiles_per_split;
    const int kt_end = min(total_k_tiles, kt_begin + args.k_tiles_per_split);
    const int n_kt = max(0, kt_end - kt_begin);
    constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(acc_bar, 1);
        abort_flag->value = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (n_kt > 0) {
        if (warp == 0) {
            if (elect_one()) {
                for (int i = 0; i < n_kt; ++i) {
                    const int s = i % STAGES;
                    const uint32_t ph = (i / STAGES) & 1;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1, abort_flag, args.status, 0x100)) break;
                    uint8_t* sa = smem + s * L::kStageBytes;
                    uint8_t* sb = sa + L::kABytes;
                    mbar_arrive_expect_tx(&full_bar[s], L::kStageBytes);
                    const int k0 = (kt_begin + i) * 64;
                    if (A_MN) {   // global A is [K rows, M contiguous]: two slabs of 64 K-rows x 64 M
                        tma_load_2d(sa, &tmap_a, &full_bar[s], m0, k0);
                        tma_load_2d(sa + 8192, &tmap_a, &full_bar[s], m0 + 64, k0);
                    } else {      // global A is [M rows, K contiguous]: one slab of 128 rows x 64 K
                        tma_load_2d(sa, &tmap_a, &full_bar[s], k0, m0);
                    }
                    if (B_MN) {
                        for (int j = 0; j < BN / 64; ++j)
                            tma_load_2d(sb + j * 8192, &tmap_b, &full_bar[s], n0 + j * 64, k0);
                    } else {
                        tma_load_2d(sb, &tmap_b, &full_bar[s], k0, n0);
                    }
                }
            }
        } else if (warp == 1) {
            if (elect_one()) {
                constexpr uint32_t idesc = make_idesc_bf16(128, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
                bool ok = true;
                for (int i = 0; i < n_kt && ok; ++i) {
                    const int s = i % STAGES;
                    const uint32_t ph = (i / STAGES) & 1;
                    ok = mbar_wait(&full_bar[s], ph, abort_flag, args.status, 0x200);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_u32(smem + s * L::kStageBytes);
                    const uint32_t sb = sa + L::kABytes;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t da = A_MN ? desc_mn_major(sa + k * 2048, 8192) : desc_k_major(sa + k * 32);
                        const uint64_t db = B_MN ? desc_mn_major(sb + k * 2048, 8192) : desc_k_major(sb + k * 32);
                        mma_ss(tmem_base, da, db, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(&empty_bar[s]);
                }
                mma_commit(acc_bar);
            }
        } else {
            // Epilogue: TMEM lane = output row within the tile, TMEM column = output column.
            const int quarter = warp & 3;
            const int row = m0 + quarter * 32 + lane;
            if (mbar_wait_warp(acc_bar, 0, abort_flag, args.status, 0x300)) {
                tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld_x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + c * 32, r);
                    tmem_ld_wait();
                    if (row < args.M) {
                        if (EPI == EPI_BF16) {
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(args.C) +
                                                 static_cast<size_t>(row) * args.ldc + n0 + c * 32;
                            uint4* dst4 = reinterpret_cast<uint4*>(dst);
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
                            float* dst = reinterpret_cast<float*>(args.C) + static_cast<size_t>(row) * args.ldc +
                                         n0 + c * 32;
#pragma unroll
                            for (int v = 0; v < 32; ++v) atomicAdd(dst + v, __uint_as_float(r[v]));
                        }
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, kTmemCols); }
}

}  // namespace laga
