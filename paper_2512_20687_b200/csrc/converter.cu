// Context converter U^(l) (Section 2.1.2): U[b, n] = sum_k x[b,k] W[k,n] (+ bias[n]),
// n = r*D + j for prefix r, feature j.
#include "common.cuh"

namespace {

// Shared-memory tiled product: a CTA computes a [16 x 64] tile of U.
__global__ void __launch_bounds__(256)
converter_tile_kernel(const ConvParams p) {
    __shared__ float xs[16][65];
    __shared__ float ws[64][65];                  // ws[k][n]
    const int n0 = blockIdx.x * 64, b0 = blockIdx.y * 16;
    const int tn = threadIdx.x & 63, tb = threadIdx.x >> 6;     // 4 rows of 16 per thread: tb, tb+4, ...
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = 0; k0 < p.D; k0 += 64) {
        for (int t = threadIdx.x; t < 16 * 64; t += 256) {
            const int b = t >> 6, k = t & 63;
            xs[b][k] = (b0 + b < p.B) ? __bfloat162float(p.x[(size_t)(b0 + b) * p.D + k0 + k]) : 0.f;
        }
        for (int t = threadIdx.x; t < 64 * 64; t += 256) {
            if (p.w_out_major) {                  // W[n][k]: k contiguous
                const int n = t >> 6, k = t & 63;
                ws[k][n] = __bfloat162float(p.w[(size_t)(n0 + n) * p.D + k0 + k]);
            } else {                              // W[k][n]: n contiguous
                const int k = t >> 6, n = t & 63;
                ws[k][n] = __bfloat162float(p.w[(size_t)(k0 + k) * p.N + n0 + n]);
            }
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < 64; ++k) {
            const float w = ws[k][tn];
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] += xs[tb + 4 * j][k] * w;
        }
        __syncthreads();
    }
    const float bias = p.bias ? __bfloat162float(p.bias[n0 + tn]) : 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int b = b0 + tb + 4 * j;
        if (b < p.B) p.U[(size_t)b * p.N + n0 + tn] = __float2bfloat16_rn(acc[j] + bias);
    }
}

}  // namespace

cudaError_t launch_converter(photon_ctx *, const ConvParams &p, cudaStream_t st,
                             long long *launches) {
    if (p.B == 0) return cudaSuccess;
    dim3 grid(p.N / 64, (p.B + 15) / 16);
    converter_tile_kernel<<<grid, 256, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}
