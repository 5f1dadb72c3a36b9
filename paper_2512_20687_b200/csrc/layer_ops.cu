// The two element-wise steps of a LLaMA layer around the attention of STEP
// (Eq. 12; all models are LLaMA Transformers, Section 3.1):
//  * rope_split_kernel: takes the fused projection qkv [n, (Hq + 2 Hkv) dh] apart
//    into q [n, Hq, dh], k [n, Hkv, dh], v [n, Hkv, dh] (the layouts the append and
//    the attention read) and rotates every head of q and k by the item's position
//    (its cache length before the append), half-split pairing, base theta; for the
//    STEP of a whole layer the same kernel writes k and v straight into the cache
//    row and updates the length (no k/v intermediate, no separate append launch);
//  * swiglu_kernel: out = silu(gate) * up for gu [n, 2F] = [gate | up].
// Both are tiny and bound by launch and memory latency: 16-byte accesses, one
// rounding to bf16 at the output.  The angles are computed in double precision
// per item and reduced to [-pi, pi] there (positions reach thousands of
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

// Where the rotated keys and the values of item i go when the split also appends (STEP of a layer:
// item i is unit i of the cache, its position is the unit's length, which grows by one).
struct AppendTo {
    bf16 *k, *v;
    int32_t *len;
    int cap;
    Paging pg;
    int32_t *status;
};

// Items are dealt to the CTAs round-robin.  The sines and cosines of an item are shared by all its
// heads through shared memory; the table of a CTA's next item (and the position of the one after)
// is prepared while the current item's data is in flight, so one barrier per item is all the
// synchronisation there is.  The inverse wavelengths do not depend on the item: once per thread.
// APPEND: k and v rows are written into the cache at row len[i] instead of k_out / v_out, with the
// checks of the append kernel (a full cache or a bad page sets the status bit, leaves the cache
// and the length alone; q is written all the same).  A length is read at least one barrier before
// the one thread that updates it writes, and no other CTA touches that unit.
template <bool APPEND>
__global__ void __launch_bounds__(EW_THREADS)
rope_split_kernel(const bf16 *qkv, const int32_t *pos, int period, int n, int Hq, int Hkv, int dh, double log2_theta,
                  bf16 *q, bf16 *k_out, bf16 *v_out, const AppendTo to) {
    __shared__ __align__(16) float cs[2][128], sn[2][128];
    const int half = dh / 2, vec_half = half / 8;        // 16-byte pieces per half head
    const int j0 = (threadIdx.x % vec_half) * 8;         // 256 is a multiple of vec_half: the same features for every piece
    const double inv = exp2(-2.0 * (double)threadIdx.x / dh * log2_theta);
    const int rotated = (Hq + Hkv) * vec_half, copied = Hkv * dh / 8;
    const int width = (Hq + 2 * Hkv) * dh, step = gridDim.x;
    ptx::grid_dep_wait();                   // qkv is the output of the kernel before this one
    // The appending form must not let the next kernel start early: it reads and then updates the lengths, so an SM
    // can hold a line of len[] in L1 in which only its own unit is current, and the attention that follows reads
    // the lengths through the read-only path.  Launched after this grid has ended (as after the append kernel, which
    // never releases its dependents early either) the attention starts with a clean L1.
    if (!APPEND) ptx::grid_dep_launch();
    auto where = [&](int i) { return i < n ? (pos ? pos[i] : i % period) : 0; };   // no position array: row i % period of its group
    auto table = [&](int at, int buf) {
        // the angle and its reduction to [-pi, pi] in double precision, sine and cosine of the remainder in single
        const double a = (double)at * inv;
        const double turns = rint(a * 0.15915494309189535);
        __sincosf((float)fma(turns, -6.283185307179586, a), &sn[buf][threadIdx.x], &cs[buf][threadIdx.x]);
    };
    const bool tabler = (int)threadIdx.x < half;
    int at = where(blockIdx.x), at_next = where(blockIdx.x + step);
    if (tabler) table(at, 0);
    __syncthreads();
    int buf = 0;
    for (int i = blockIdx.x; i < n; i += step, buf ^= 1) {
        const bf16 *row = qkv + (size_t)i * width;
        const int at_after = where(i + 2 * step);         // in flight under this item's work
        // rows of the [Hkv, dh] slices of k and v that belong to this item
        bf16 *kd = k_out + (size_t)i * Hkv * dh, *vd = v_out + (size_t)i * Hkv * dh;
        size_t head_stride = dh;
        bool keep = true;
        if (APPEND) {
            keep = at >= 0 && at < to.cap;
            if (!keep && threadIdx.x == 0) atomicOr(to.status, PHOTON_DEV_CAPACITY);
            size_t first = ((size_t)i * Hkv * to.cap + at) * dh;
            head_stride = (size_t)to.cap * dh;
            if (keep && to.pg.table) {
                const int id = to.pg.table[(size_t)i * to.pg.pages_per_unit + at / to.pg.page_rows];
                keep = id >= 0 && id < to.pg.n_pages;
                if (!keep && threadIdx.x == 0) atomicOr(to.status, PHOTON_DEV_BAD_INDEX);
                first = ((size_t)id * Hkv * to.pg.page_rows + at % to.pg.page_rows) * dh;
                head_stride = (size_t)to.pg.page_rows * dh;
            }
            if (!keep) first = 0;
            kd = to.k + first;
            vd = to.v + first;
        }
        // piece p of head h covers features [8p, 8p + 8) and their partners 8p + half ..
        for (int w0 = 0; w0 < rotated + copied; w0 += EW_THREADS) {
            const int w = w0 + threadIdx.x;
            uint4 ua = {}, ub = {};
            const int h = w / vec_half;
            if (w < rotated) {
                ua = *reinterpret_cast<const uint4 *>(row + (size_t)h * dh + j0);
                ub = *reinterpret_cast<const uint4 *>(row + (size_t)h * dh + j0 + half);
            } else if (w < rotated + copied) {
                ua = reinterpret_cast<const uint4 *>(row + (size_t)(Hq + Hkv) * dh)[w - rotated];
            }
            if (w0 == 0 && tabler) table(at_next, buf ^ 1);      // under the loads: the next item's table
            if (w < rotated) {
                bf16 *o = h < Hq ? q + ((size_t)i * Hq + h) * dh : kd + (size_t)(h - Hq) * head_stride;
                float a[8], b[8], c[8], s[8], ra[8], rb[8];
                unpack8(ua, a);
                unpack8(ub, b);
                *reinterpret_cast<float4 *>(c) = *reinterpret_cast<const float4 *>(&cs[buf][j0]);
                *reinterpret_cast<float4 *>(c + 4) = *reinterpret_cast<const float4 *>(&cs[buf][j0 + 4]);
                *reinterpret_cast<float4 *>(s) = *reinterpret_cast<const float4 *>(&sn[buf][j0]);
                *reinterpret_cast<float4 *>(s + 4) = *reinterpret_cast<const float4 *>(&sn[buf][j0 + 4]);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    ra[e] = a[e] * c[e] - b[e] * s[e];
                    rb[e] = b[e] * c[e] + a[e] * s[e];
                }
                if (h < Hq || keep) {
                    *reinterpret_cast<uint4 *>(o + j0) = pack8(ra);
                    *reinterpret_cast<uint4 *>(o + j0 + half) = pack8(rb);
                }
            } else if (w < rotated + copied && keep) {
                const int piece = w - rotated, per_head = dh / 8;
                *reinterpret_cast<uint4 *>(vd + (size_t)(piece / per_head) * head_stride + (piece % per_head) * 8) = ua;
            }
        }
        __syncthreads();
        if (APPEND && keep && threadIdx.x == 0) to.len[i] = at + 1;
        at = at_next;
        at_next = at_after;
    }
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
    const cudaError_t e = launch_dependent(rope_split_kernel<false>, dim3(std::min(n, 148 * 8)), dim3(EW_THREADS), 0, st, 0, qkv, pos,
                                           period, n, Hq, Hkv, dh, log2((double)theta), q, k, v, AppendTo{});
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_rope_split_append(const bf16 *qkv, int n, int Hq, int Hkv, int dh, float theta, bf16 *q, bf16 *k_cache,
                                     bf16 *v_cache, int32_t *len, int cap, Paging pg, int32_t *status, cudaStream_t st,
                                     long long *launches) {
    if (n == 0) return cudaSuccess;
    const cudaError_t e = launch_dependent(rope_split_kernel<true>, dim3(std::min(n, 148 * 8)), dim3(EW_THREADS), 0, st, 0, qkv,
                                           (const int32_t *)len, 1, n, Hq, Hkv, dh, log2((double)theta), q, (bf16 *)nullptr,
                                           (bf16 *)nullptr, AppendTo{k_cache, v_cache, len, cap, pg, status});
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
