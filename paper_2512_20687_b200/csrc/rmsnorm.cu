// Root-mean-square normalisation of rows with a learned per-feature scale: the
// first half of the top-level context chunker (Section 2.1.1), whose input is
// the concatenation of the C_L lower-level latents of a meta-context:
//   out[r, c] = x[r, c] * gamma[c] / sqrt(mean_c x[r, c]^2 + eps).
// One CTA per row, 16-byte loads, fp32 sums, one rounding to bf16 at the output
// (what the linear half reads).  Rows are a few KB: the second pass over a row
// comes from L1/L2.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int RN_THREADS = 256;

__global__ void __launch_bounds__(RN_THREADS)
rmsnorm_kernel(const bf16 *x, const bf16 *gamma, float eps, bf16 *out, int cols) {
    __shared__ float part[RN_THREADS / 32];
    ptx::grid_dep_wait();                   // x may be the output of the kernel before this one
    ptx::grid_dep_launch();
    const uint4 *row = reinterpret_cast<const uint4 *>(x + (size_t)blockIdx.x * cols);
    const int n_vec = cols / 8;
    float ss = 0.f;
    for (int i = threadIdx.x; i < n_vec; i += RN_THREADS) {
        const uint4 v = row[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float a = bf16_lo(w[e]), b = bf16_hi(w[e]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < RN_THREADS / 32; ++w) tot += part[w];       // same order in every thread
    const float inv = rsqrtf(tot / (float)cols + eps);
    uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)blockIdx.x * cols);
    const uint4 *gv = reinterpret_cast<const uint4 *>(gamma);
    for (int i = threadIdx.x; i < n_vec; i += RN_THREADS) {
        const uint4 v = row[i];
        const uint4 g = gamma ? gv[i] : make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);   // ones
        const uint32_t w[4] = {v.x, v.y, v.z, v.w}, gw[4] = {g.x, g.y, g.z, g.w};
        uint32_t r[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 t = __floats2bfloat162_rn(bf16_lo(w[e]) * bf16_lo(gw[e]) * inv,
                                                     bf16_hi(w[e]) * bf16_hi(gw[e]) * inv);
            r[e] = *reinterpret_cast<uint32_t *>(&t);
        }
        dst[i] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

}  // namespace

cudaError_t launch_rmsnorm(const bf16 *x, const bf16 *gamma, float eps, bf16 *out, int rows, int cols,
                           cudaStream_t st, long long *launches) {
    if (rows == 0) return cudaSuccess;
    const cudaError_t e = launch_dependent(rmsnorm_kernel, dim3(rows), dim3(RN_THREADS), 0, st, 0, x, gamma, eps, out, cols);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}
