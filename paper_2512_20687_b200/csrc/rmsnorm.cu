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

// Rows of at most 2048 columns: a warp per row, the row held in registers between the sum and the scaling
// (one read), no CTA-wide barrier.
constexpr int RN_MAXV = 8;                  // 16-byte pieces per lane: 32 * 8 * 8 = 2048 columns

__global__ void __launch_bounds__(RN_THREADS)
rmsnorm_rows_kernel(const bf16 *x, const bf16 *gamma, float eps, bf16 *out, int rows, int cols) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (RN_THREADS / 32) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const int n_vec = cols / 8;
    const uint4 *row = reinterpret_cast<const uint4 *>(x + (size_t)r * cols);
    uint4 v[RN_MAXV];
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < RN_MAXV; ++t) {
        const int i = lane + 32 * t;
        v[t] = i < n_vec ? row[i] : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t w[4] = {v[t].x, v[t].y, v[t].z, v[t].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float a = bf16_lo(w[e]), b = bf16_hi(w[e]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float inv = rsqrtf(ss / (float)cols + eps);
    uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)r * cols);
    const uint4 *gv = reinterpret_cast<const uint4 *>(gamma);
#pragma unroll
    for (int t = 0; t < RN_MAXV; ++t) {
        const int i = lane + 32 * t;
        if (i >= n_vec) continue;
        const uint4 g = gamma ? gv[i] : make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);   // ones
        const uint32_t w[4] = {v[t].x, v[t].y, v[t].z, v[t].w}, gw[4] = {g.x, g.y, g.z, g.w};
        uint32_t o4[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 q = __floats2bfloat162_rn(bf16_lo(w[e]) * bf16_lo(gw[e]) * inv,
                                                     bf16_hi(w[e]) * bf16_hi(gw[e]) * inv);
            o4[e] = *reinterpret_cast<uint32_t *>(&q);
        }
        dst[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
    }
}

}  // namespace

cudaError_t launch_rmsnorm(const bf16 *x, const bf16 *gamma, float eps, bf16 *out, int rows, int cols,
                           cudaStream_t st, long long *launches) {
    if (rows == 0) return cudaSuccess;
    const int per_cta = RN_THREADS / 32;
    const cudaError_t e =
        cols <= RN_MAXV * 256 && rows >= 1024           // enough rows for a warp per row to fill the GPU
            ? launch_dependent(rmsnorm_rows_kernel, dim3((rows + per_cta - 1) / per_cta), dim3(RN_THREADS), 0, st, 0, x, gamma,
                               eps, out, rows, cols)
            : launch_dependent(rmsnorm_kernel, dim3(rows), dim3(RN_THREADS), 0, st, 0, x, gamma, eps, out, cols);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}
