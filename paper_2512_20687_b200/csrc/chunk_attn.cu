// Chunk-local bounded attention of the local decoders (Eq. 6-7): every query
// attends the first len rows of its own chunk buffer only.
#include <math_constants.h>

#include "common.cuh"

namespace {

// part p of a query covers: p < splits_sh ? a range of the shared segment : a range of its own rows
__device__ __forceinline__ void part_range(int L, int n_splits, int p, int &r0, int &r1) {
    const int per = (L + n_splits - 1) / n_splits;
    r0 = min(L, p * per);
    r1 = min(L, r0 + per);
}

// One warp per (query, query head, part).  Lane l owns elements
// [l*DH/32, (l+1)*DH/32) of every row.
template <int DH>
__global__ void __launch_bounds__(128)
attn_partial_kernel(const AttnParams p) {
    constexpr int E = DH / 32;                 // elements per lane (2 or 4)
    const int parts = p.splits_sh + p.splits_own;
    const long long wid = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    const long long total = (long long)p.n_q * p.Hq * parts;
    if (wid >= total) return;
    const int lane = threadIdx.x & 31;
    const int part = (int)(wid % parts);
    const int hq = (int)((wid / parts) % p.Hq);
    const int i = (int)(wid / ((long long)parts * p.Hq));
    const int kvh = hq / (p.Hq / p.Hkv);

    float *dst = p.partials + (size_t)wid * (DH + 2);
    const int u = p.slot ? p.slot[i] : i;
    const bf16 *kb = nullptr, *vb = nullptr;
    int r0 = 0, r1 = 0;
    bool bad = (u < 0 || u >= p.n_units);
    if (!bad) {
        if (part < p.splits_sh) {
            const int s = p.sh_id ? p.sh_id[u] : -1;
            if (s >= p.n_shared) bad = true;
            else if (s >= 0) {
                part_range(p.sh_len[s], p.splits_sh, part, r0, r1);
                const size_t base = ((size_t)s * p.Hkv + kvh) * p.cap_sh * DH;
                kb = p.ks + base; vb = p.vs + base;
            }
        } else {
            // a bad shared id voids the whole query, own parts included
            const int s = (p.sh_id && p.splits_sh) ? p.sh_id[u] : -1;
            if (s >= p.n_shared) bad = true;
            else {
                part_range(min(p.len[u], p.cap), p.splits_own, part - p.splits_sh, r0, r1);
                const size_t base = ((size_t)u * p.Hkv + kvh) * p.cap * DH;
                kb = p.k + base; vb = p.v + base;
            }
        }
    }
    if (bad) {
        if (lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
        r0 = r1 = 0;
    }

    float qf[E];
    {
        const bf16 *qp = p.q + ((size_t)i * p.Hq + hq) * DH + lane * E;
#pragma unroll
        for (int e = 0; e < E; ++e) qf[e] = __bfloat162float(qp[e]) * p.scale_log2;
    }
    float m = -CUDART_INF_F, l = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;

    for (int r = r0; r < r1; ++r) {
        const bf16 *kr = kb + (size_t)r * DH + lane * E;
        const bf16 *vr = vb + (size_t)r * DH + lane * E;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) s += qf[e] * __bfloat162float(kr[e]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float mn = fmaxf(m, s);
        const float corr = exp2f(m - mn);          // m = -inf on the first key: exp2(-inf) = 0
        const float w = exp2f(s - mn);
        l = l * corr + w;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + w * __bfloat162float(vr[e]);
        m = mn;
    }
#pragma unroll
    for (int e = 0; e < E; ++e) dst[lane * E + e] = acc[e];
    if (lane == 0) { dst[DH] = m; dst[DH + 1] = l; }
}

// One warp per (query, query head): log-sum-exp combination of its parts.
template <int DH>
__global__ void __launch_bounds__(128)
attn_merge_kernel(const AttnParams p) {
    constexpr int E = DH / 32;
    const int parts = p.splits_sh + p.splits_own;
    const long long wid = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (wid >= (long long)p.n_q * p.Hq) return;
    const int lane = threadIdx.x & 31;
    const float *src = p.partials + (size_t)wid * parts * (DH + 2);
    float M = -CUDART_INF_F;
    for (int j = 0; j < parts; ++j) M = fmaxf(M, src[(size_t)j * (DH + 2) + DH]);
    float L = 0.f, o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = 0.f;
    for (int j = 0; j < parts; ++j) {
        const float *pj = src + (size_t)j * (DH + 2);
        const float lj = pj[DH + 1];
        if (lj == 0.f) continue;                    // empty part
        const float w = exp2f(pj[DH] - M);
        L += lj * w;
#pragma unroll
        for (int e = 0; e < E; ++e) o[e] += w * pj[lane * E + e];
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    bf16 *op = p.out + (size_t)wid * DH + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) op[e] = __float2bfloat16_rn(o[e] * inv);
    if (p.lse && lane == 0)
        p.lse[wid] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -CUDART_INF_F;
}

template <int DH>
cudaError_t run(const AttnParams &p, cudaStream_t st, long long *launches) {
    if (p.n_q == 0) return cudaSuccess;
    const int parts = p.splits_sh + p.splits_own;
    const long long warps = (long long)p.n_q * p.Hq * parts;
    attn_partial_kernel<DH><<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(p);
    const long long mw = (long long)p.n_q * p.Hq;
    attn_merge_kernel<DH><<<(unsigned)((mw + 3) / 4), 128, 0, st>>>(p);
    *launches += 2;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_chunk_attention(photon_ctx *, const AttnParams &p, cudaStream_t st,
                                   long long *launches) {
    return p.dh == 64 ? run<64>(p, st, launches) : run<128>(p, st, launches);
}
