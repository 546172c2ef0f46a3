// RMS normalisation over the head dimension with its forward-mode tangent, one pass over HBM.
//
// DiT attention blocks normalise q and k per head before the scores are formed (Sec. 3.1, "QK normalization");
// in JVP mode the layer must hand the attention kernel both the normalised primal and its tangent
// (Appendix C.2 restructures an RMSNorm layer this way with PyTorch's forward-mode operator).  For one row
// x in R^D with frozen weight w (the JVP runs on the stop-gradient network, Algorithm 1 line 4):
//     n  = sqrt(mean(x^2) + eps)
//     y  = w . x / n
//     ty = w . (tx / n - x (x . tx) / (D n^3))
// Memory bound: 2 reads + 2 writes of D bf16 per row.  D/8 threads own a row (16-byte accesses, so a row
// of D = 128 is two fully used 128-byte lines per tensor), sums go through warp shuffles, the grid is a
// multiple of the SM count and strides over the rows.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace attn_jvp {

template <int D, bool kHasTangent>
__global__ void __launch_bounds__(256)
qknorm_jvp_kernel(const uint4* __restrict__ x, const uint4* __restrict__ tx, const float* __restrict__ w,
                  uint4* __restrict__ y, uint4* __restrict__ ty, long long rows, float eps) {
    constexpr int kLanesPerRow = D / 8;                       // 16 (D = 128) or 8 (D = 64)
    constexpr int kRowsPerBlock = 256 / kLanesPerRow;
    const int sub = threadIdx.x % kLanesPerRow;              // which 8-element piece of the row
    const int row_in_block = threadIdx.x / kLanesPerRow;
    float wv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) wv[i] = w[sub * 8 + i];

    // The loop bound is the same for every thread of the block (the shuffles below need whole warps); a thread
    // whose row is past the end works on the last row and stores nothing.
    for (long long base = static_cast<long long>(blockIdx.x) * kRowsPerBlock; base < rows;
         base += static_cast<long long>(gridDim.x) * kRowsPerBlock) {
        const long long r_own = base + row_in_block;
        const bool active = r_own < rows;
        const long long r = active ? r_own : rows - 1;
        const long long idx = r * kLanesPerRow + sub;
        const uint4 xr = x[idx];
        uint4 tr = make_uint4(0u, 0u, 0u, 0u);
        if (kHasTangent) tr = tx[idx];
        float xv[8], tv[8];
        const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
        const uint32_t tw[4] = {tr.x, tr.y, tr.z, tr.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            xv[2 * i] = __uint_as_float(xw[i] << 16);          // bf16 -> fp32 is a shift
            xv[2 * i + 1] = __uint_as_float(xw[i] & 0xFFFF0000u);
            tv[2 * i] = __uint_as_float(tw[i] << 16);
            tv[2 * i + 1] = __uint_as_float(tw[i] & 0xFFFF0000u);
        }
        float ss = 0.0f, st = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            ss = fmaf(xv[i], xv[i], ss);
            st = fmaf(xv[i], tv[i], st);
        }
#pragma unroll
        for (int m = kLanesPerRow / 2; m >= 1; m >>= 1) {
            ss += __shfl_xor_sync(0xffffffffu, ss, m);
            if (kHasTangent) st += __shfl_xor_sync(0xffffffffu, st, m);
        }
        const float inv_n = rsqrtf(ss * (1.0f / D) + eps);
        const float coef = st * (1.0f / D) * inv_n * inv_n * inv_n;      // (x . tx) / (D n^3)
        uint32_t yo[4], to[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float y0 = wv[2 * i] * xv[2 * i] * inv_n, y1 = wv[2 * i + 1] * xv[2 * i + 1] * inv_n;
            __nv_bfloat162 hy = __floats2bfloat162_rn(y0, y1);
            yo[i] = *reinterpret_cast<uint32_t*>(&hy);
            if (kHasTangent) {
                const float t0 = wv[2 * i] * fmaf(tv[2 * i], inv_n, -xv[2 * i] * coef);
                const float t1 = wv[2 * i + 1] * fmaf(tv[2 * i + 1], inv_n, -xv[2 * i + 1] * coef);
                __nv_bfloat162 ht = __floats2bfloat162_rn(t0, t1);
                to[i] = *reinterpret_cast<uint32_t*>(&ht);
            }
        }
        if (active) {
            y[idx] = make_uint4(yo[0], yo[1], yo[2], yo[3]);
            if (kHasTangent) ty[idx] = make_uint4(to[0], to[1], to[2], to[3]);
        }
    }
}

}  // namespace attn_jvp
