// The two element-wise steps of a LLaMA layer around the attention of STEP
// (Eq. 12; all models are LLaMA Transformers, Section 3.1):
//  * rope_split_kernel: takes the fused projection qkv [n, (Hq + 2 Hkv) dh] apart
//    into q [n, Hq, dh], k [n, Hkv, dh], v [n, Hkv, dh] (the layouts the append and
//    the attention read) and rotates every head of q and k by the item's position
//    (its cache length before the append), half-split pairing, base theta;
//  * swiglu_kernel: out = silu(gate) * up for gu [n, 2F] = [gate | up].
// Both are tiny and bound by launch and memory latency: 16-byte accesses, one
// rounding to bf16 at the output.  The angles are computed in double precision
// once per item and reduced to [-pi, pi] there (positions reach thousands of
// radians, which single-precision sines do not survive); the remainder goes
// through the fast single-precision sine and cosine, and all heads share the
// table through shared memory.
#include <algorithm>
#include <cmath>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int EW_THREADS = 256;

__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8]) {
    f[0] = bf16_lo(u.x); f[1] = bf16_hi(u.x); f[2] = bf16_lo(u.y); f[3] = bf16_hi(u.y);
    f[4] = bf16_lo(u.z); f[5] = bf16_hi(u.z); f[6] = bf16_lo(u.w); f[7] = bf16_hi(u.w);
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
    uint4 u;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(f[0], f[1]); u.x = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[2], f[3]); u.y = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[4], f[5]); u.z = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[6], f[7]); u.w = *reinterpret_cast<uint32_t *>(&t);
    return u;
}

// one CTA per item; dh <= 256
__global__ void __launch_bounds__(EW_THREADS)
rope_split_kernel(const bf16 *qkv, const int32_t *pos, int period, int Hq, int Hkv, int dh, double log2_theta,
                  bf16 *q, bf16 *k, bf16 *v) {
    __shared__ float cs[128], sn[128];
    ptx::grid_dep_wait();                   // qkv is the output of the kernel before this one
    ptx::grid_dep_launch();
    const int i = blockIdx.x, half = dh / 2;
    const int at = pos ? pos[i] : i % period;          // no position array: item i is row i % period of its group
    for (int j = threadIdx.x; j < half; j += EW_THREADS) {
        // the angle and its reduction to [-pi, pi] in double precision, sine and cosine of the remainder in single
        const double a = (double)at * exp2(-2.0 * j / dh * log2_theta);
        const double turns = rint(a * 0.15915494309189535);
        const float r = (float)fma(turns, -6.283185307179586, a);
        float s, c;
        __sincosf(r, &s, &c);
        cs[j] = c; sn[j] = s;
    }
    __syncthreads();
    const int width = (Hq + 2 * Hkv) * dh;
    const bf16 *row = qkv + (size_t)i * width;
    const int vec_half = half / 8;                       // 16-byte pieces per half head
    // rotated heads: piece p of head h covers features [8p, 8p + 8) and their partners 8p + half ..
    for (int w = threadIdx.x; w < (Hq + Hkv) * vec_half; w += EW_THREADS) {
        const int h = w / vec_half, j0 = (w % vec_half) * 8;
        const bf16 *x = row + (size_t)h * dh;
        bf16 *o = h < Hq ? q + ((size_t)i * Hq + h) * dh : k + ((size_t)i * Hkv + (h - Hq)) * dh;
        float a[8], b[8], ra[8], rb[8];
        unpack8(*reinterpret_cast<const uint4 *>(x + j0), a);
        unpack8(*reinterpret_cast<const uint4 *>(x + j0 + half), b);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float c = cs[j0 + e], s = sn[j0 + e];
            ra[e] = a[e] * c - b[e] * s;
            rb[e] = b[e] * c + a[e] * s;
        }
        *reinterpret_cast<uint4 *>(o + j0) = pack8(ra);
        *reinterpret_cast<uint4 *>(o + j0 + half) = pack8(rb);
    }
    const uint4 *vs = reinterpret_cast<const uint4 *>(row + (size_t)(Hq + Hkv) * dh);
    uint4 *vd = reinterpret_cast<uint4 *>(v + (size_t)i * Hkv * dh);
    for (int w = threadIdx.x; w < Hkv * dh / 8; w += EW_THREADS) vd[w] = vs[w];
}

__global__ void __launch_bounds__(EW_THREADS)
swiglu_kernel(const bf16 *gu, bf16 *out, int n, int F) {
    ptx::grid_dep_wait();
    ptx::grid_dep_launch();
    const int per_row = F / 8;
    const long long total = (long long)n * per_row;
    for (long long w = (long long)blockIdx.x * EW_THREADS + threadIdx.x; w < total; w += (long long)gridDim.x * EW_THREADS) {
        const long long i = w / per_row;
        const int f0 = (int)(w % per_row) * 8;
        float g[8], u[8], r[8];
        unpack8(*reinterpret_cast<const uint4 *>(gu + i * 2 * F + f0), g);
        unpack8(*reinterpret_cast<const uint4 *>(gu + i * 2 * F + F + f0), u);
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = g[e] / (1.f + __expf(-g[e])) * u[e];
        *reinterpret_cast<uint4 *>(out + i * F + f0) = pack8(r);
    }
}

}  // namespace

cudaError_t launch_rope_split(const bf16 *qkv, const int32_t *pos, int period, int n, int Hq, int Hkv, int dh,
                              float theta, bf16 *q, bf16 *k, bf16 *v, cudaStream_t st, long long *launches) {
    if (n == 0) return cudaSuccess;
    const cudaError_t e = launch_dependent(rope_split_kernel, dim3(n), dim3(EW_THREADS), 0, st, 0, qkv, pos, period, Hq, Hkv, dh,
                                           log2((double)theta), q, k, v);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_swiglu(const bf16 *gu, bf16 *out, int n, int F, cudaStream_t st, long long *launches) {
    if (n == 0) return cudaSuccess;
    const long long vecs = (long long)n * (F / 8);
    const unsigned grid = (unsigned)std::min<long long>((vecs + EW_THREADS - 1) / EW_THREADS, 148 * 8);
    const cudaError_t e = launch_dependent(swiglu_kernel, dim3(grid), dim3(EW_THREADS), 0, st, 0, gu, out, n, F);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}
