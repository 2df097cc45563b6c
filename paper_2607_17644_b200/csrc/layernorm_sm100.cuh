// LayerNorm of the latent (Algorithm 1 step 1: latent <- LayerNorm(latent), applied to the d_kv-wide output of
// W_kv_a before the sequence all-gather), forward and backward.
//
//   y[m, :]  = (x[m, :] - mean_m) * rstd_m * gamma + beta,     mean_m = sum_c x[m, c] / D,
//                                                              rstd_m = 1 / sqrt(sum_c (x[m, c] - mean_m)^2 / D + eps)
//   dx[m, :] = rstd_m * (g - mean_c(g) - xhat * mean_c(g * xhat)),   g = dy * gamma, xhat = (x - mean_m) * rstd_m
//   dgamma   = sum_m dy[m, :] * xhat[m, :],    dbeta = sum_m dy[m, :]
//
// Rows are a kilobyte (D = 512 bf16): the work is one read and one write of every element, so these kernels
// are bound by HBM and built for that -- one warp per row, 16-byte loads and stores (a lane owns 8 consecutive
// channels of every 256), all arithmetic in fp32 registers, the row statistics by warp shuffles, no shared
// memory in the forward.  The backward's column sums (dgamma, dbeta) are kept per lane in registers over all
// the rows a warp walks, combined across the block's warps in shared memory and added to the fp32 outputs
// with one atomic per channel and block; the grid is a few blocks per SM striding over the rows.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace laga {

constexpr int kLnMaxD = 1024;                 // a lane holds D / 32 values in registers
constexpr int kLnWarps = 8;
// The kernels are templated on kLnChunks = ceil(D / 256), the 16-byte chunks a lane holds per row (1, 2 or 4):
// registers, and with them the blocks resident per SM and the bytes in flight, follow the real width.

__device__ __forceinline__ void ln_unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[k]));
        f[2 * k] = t.x;
        f[2 * k + 1] = t.y;
    }
}
__device__ __forceinline__ uint4 ln_pack(const float* f) {
    uint4 v;
    uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
        w[k] = *reinterpret_cast<const uint32_t*>(&t);
    }
    return v;
}
__device__ __forceinline__ float ln_warp_sum(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// One warp per row; the grid strides over the rows.  gamma and beta are re-read for every row (2 KB that never
// leave L1) instead of being held in registers: what these kernels need is warps in flight, i.e. few registers.
template <int kLnChunks>
__global__ void __launch_bounds__(kLnWarps * 32)
layernorm_fwd_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gamma,
                     const __nv_bfloat16* __restrict__ beta, int M, int D, float eps, __nv_bfloat16* __restrict__ y,
                     float* __restrict__ mean_out, float* __restrict__ rstd_out) {
    const int lane = threadIdx.x & 31;
    const int warp_global = blockIdx.x * kLnWarps + (threadIdx.x >> 5);
    const int n_warps = gridDim.x * kLnWarps;
    const float inv_d = 1.0f / static_cast<float>(D);
    for (int m = warp_global; m < M; m += n_warps) {
        const __nv_bfloat16* row = x + static_cast<size_t>(m) * D;
        float v[kLnChunks][8];
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i) {
            const int c = i * 256 + lane * 8;
            if (c < D) {
                ln_unpack(*reinterpret_cast<const uint4*>(row + c), v[i]);
#pragma unroll
                for (int k = 0; k < 8; ++k) sum += v[i][k];
            }
        }
        const float mean = ln_warp_sum(sum) * inv_d;
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i)
            if (i * 256 + lane * 8 < D)
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float d = v[i][k] - mean;
                    sq = fmaf(d, d, sq);
                }
        const float rstd = rsqrtf(ln_warp_sum(sq) * inv_d + eps);
        __nv_bfloat16* out = y + static_cast<size_t>(m) * D;
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i) {
            const int c = i * 256 + lane * 8;
            if (c < D) {
                float gm[8], bt[8], o[8];
                ln_unpack(__ldg(reinterpret_cast<const uint4*>(gamma + c)), gm);
                if (beta != nullptr) ln_unpack(__ldg(reinterpret_cast<const uint4*>(beta + c)), bt);
#pragma unroll
                for (int k = 0; k < 8; ++k) o[k] = fmaf((v[i][k] - mean) * rstd, gm[k], beta != nullptr ? bt[k] : 0.f);
                *reinterpret_cast<uint4*>(out + c) = ln_pack(o);
            }
        }
        if (lane == 0) {
            if (mean_out != nullptr) mean_out[m] = mean;
            if (rstd_out != nullptr) rstd_out[m] = rstd;
        }
    }
}

// dgamma / dbeta must be zero when the kernel starts (the host clears them).
template <int kLnChunks>
__global__ void __launch_bounds__(kLnWarps * 32)
layernorm_bwd_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ x,
                     const __nv_bfloat16* __restrict__ gamma, const float* __restrict__ mean_in,
                     const float* __restrict__ rstd_in, int M, int D, __nv_bfloat16* __restrict__ dx,
                     float* __restrict__ dgamma, float* __restrict__ dbeta) {
    __shared__ float part[kLnWarps][kLnChunks * 256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warp_global = blockIdx.x * kLnWarps + warp;
    const int n_warps = gridDim.x * kLnWarps;
    const float inv_d = 1.0f / static_cast<float>(D);
    float acc_g[kLnChunks][8], acc_b[kLnChunks][8];
#pragma unroll
    for (int i = 0; i < kLnChunks; ++i)
#pragma unroll
        for (int k = 0; k < 8; ++k) acc_g[i][k] = acc_b[i][k] = 0.f;
    for (int m = warp_global; m < M; m += n_warps) {
        const float mean = mean_in[m], rstd = rstd_in[m];
        const __nv_bfloat16* xr = x + static_cast<size_t>(m) * D;
        const __nv_bfloat16* gr = dy + static_cast<size_t>(m) * D;
        float xh[kLnChunks][8], g[kLnChunks][8];
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i) {
            const int c = i * 256 + lane * 8;
            if (c < D) {
                float xv[8], dv[8], gm[8];
                ln_unpack(*reinterpret_cast<const uint4*>(xr + c), xv);
                ln_unpack(*reinterpret_cast<const uint4*>(gr + c), dv);
                ln_unpack(__ldg(reinterpret_cast<const uint4*>(gamma + c)), gm);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    xh[i][k] = (xv[k] - mean) * rstd;
                    g[i][k] = dv[k] * gm[k];
                    s1 += g[i][k];
                    s2 = fmaf(g[i][k], xh[i][k], s2);
                    acc_g[i][k] = fmaf(dv[k], xh[i][k], acc_g[i][k]);
                    acc_b[i][k] += dv[k];
                }
            }
        }
        s1 = ln_warp_sum(s1) * inv_d;
        s2 = ln_warp_sum(s2) * inv_d;
        __nv_bfloat16* out = dx + static_cast<size_t>(m) * D;
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i) {
            const int c = i * 256 + lane * 8;
            if (c < D) {
                float o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) o[k] = rstd * (g[i][k] - s1 - xh[i][k] * s2);
                *reinterpret_cast<uint4*>(out + c) = ln_pack(o);
            }
        }
    }
    // column sums: warps -> shared memory -> one atomic per channel and block (dgamma, then dbeta)
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        float* dst = pass == 0 ? dgamma : dbeta;
        if (dst == nullptr) continue;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kLnChunks; ++i) {
            const int c = i * 256 + lane * 8;
            if (c < D)
#pragma unroll
                for (int k = 0; k < 8; ++k) part[warp][c + k] = pass == 0 ? acc_g[i][k] : acc_b[i][k];
        }
        __syncthreads();
        for (int c = threadIdx.x; c < D; c += kLnWarps * 32) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kLnWarps; ++w) s += part[w][c];
            atomicAdd(dst + c, s);
        }
    }
}

}  // namespace laga
