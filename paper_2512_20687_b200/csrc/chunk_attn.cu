// Chunk-local bounded attention of the local decoders (Eq. 6-7): every query
// attends the first len rows of its own chunk buffer only (R_l prefix rows plus
// the in-chunk rows written so far), so a problem is at most P + C <= 64 keys.
//
// HBM-bound streaming of many tiny problems.  A warp owns one (chunk, KV head):
// the valid K and V rows of that pair are one contiguous run of len * dh * 2
// bytes each, which the warp fetches with 128-bit loads, all issued before the
// first use so that a warp keeps up to 2 * RP rows in flight; rows >= len are
// never touched.  A row is spread over dh/8 lanes; logits are reduced with
// warp shuffles, the softmax runs in the base-2 domain in fp32, and the G query
// heads of the group reuse the rows held in registers.  One launch, no
// workspace: the result is rounded once to bf16 and stored.
#include <math_constants.h>

#include "common.cuh"

namespace {

constexpr int CH_WARPS = 8;                 // (chunk, KV head) pairs per CTA

__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8]) {
    f[0] = bf16_lo(u.x); f[1] = bf16_hi(u.x); f[2] = bf16_lo(u.y); f[3] = bf16_hi(u.y);
    f[4] = bf16_lo(u.z); f[5] = bf16_hi(u.z); f[6] = bf16_lo(u.w); f[7] = bf16_hi(u.w);
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

// DH: head size; RP: rows fetched per pass (a pass covers rows [pass*RP, pass*RP + RP));
// GT: query heads evaluated together against the rows in registers.
template <int DH, int RP, int GT>
__global__ void __launch_bounds__(CH_WARPS * 32)
chunk_attn_kernel(const AttnParams p) {
    constexpr int VEC = DH / 8;             // 16-byte vectors (= lanes) per row
    constexpr int RPL = 32 / VEC;           // rows covered by one warp-wide load
    constexpr int NI = RP / RPL;            // loads per lane per pass
    static_assert(RP % RPL == 0, "pass height must be a whole number of warp loads");

    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * CH_WARPS + (threadIdx.x >> 5);
    if (item >= (long long)p.n_q * p.Hkv) return;
    const int kvh = (int)(item % p.Hkv);
    const int i = (int)(item / p.Hkv);
    const int G = p.Hq / p.Hkv;
    const int col = lane % VEC, rsub = lane / VEC;

    const int u = p.slot ? __ldcg(p.slot + i) : i;               // index arrays through the L2: another kernel may have just written them
    bf16 *out_base = p.out + ((size_t)i * p.Hq + (size_t)kvh * G) * DH + col * 8;
    if (u < 0 || u >= p.n_units) {
        if (lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
        if (rsub == 0)
            for (int g = 0; g < G; ++g)
                *reinterpret_cast<uint4 *>(out_base + (size_t)g * DH) = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    const int len = max(0, min(__ldcg(p.len + u), p.cap));
    const size_t base = ((size_t)u * p.Hkv + kvh) * p.cap * DH;
    const uint4 *kp = reinterpret_cast<const uint4 *>(p.k + base) + lane;     // row rsub, vector col
    const uint4 *vp = reinterpret_cast<const uint4 *>(p.v + base) + lane;
    const int n_pass = (len + RP - 1) / RP;

    for (int g0 = 0; g0 < G; g0 += GT) {
        float qf[GT][8];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const uint4 qv = *reinterpret_cast<const uint4 *>(
                p.q + ((size_t)i * p.Hq + (size_t)kvh * G + g0 + g) * DH + col * 8);
            unpack8(qv, qf[g]);
#pragma unroll
            for (int e = 0; e < 8; ++e) qf[g][e] *= p.scale_log2;
        }
        float m[GT], l[GT], acc[GT][8];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            m[g] = -CUDART_INF_F; l[g] = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[g][e] = 0.f;
        }

        for (int pass = 0; pass < n_pass; ++pass) {
            const int r0 = pass * RP + rsub;
            uint4 kr[NI], vr[NI];
#pragma unroll
            for (int t = 0; t < NI; ++t) {
                const bool ok = r0 + t * RPL < len;
                kr[t] = ok ? __ldg(kp + (size_t)(pass * RP + t * RPL) * VEC) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int t = 0; t < NI; ++t) {
                const bool ok = r0 + t * RPL < len;
                vr[t] = ok ? __ldg(vp + (size_t)(pass * RP + t * RPL) * VEC) : make_uint4(0u, 0u, 0u, 0u);
            }
            // logits of this lane's rows for each head of the group
            float s[GT][NI];
#pragma unroll
            for (int t = 0; t < NI; ++t) {
                float kf[8];
                unpack8(kr[t], kf);
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    float a = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) a = fmaf(qf[g][e], kf[e], a);
                    s[g][t] = a;
                }
            }
#pragma unroll
            for (int g = 0; g < GT; ++g)
#pragma unroll
                for (int t = 0; t < NI; ++t) {
#pragma unroll
                    for (int o = 1; o < VEC; o <<= 1) s[g][t] += __shfl_xor_sync(0xffffffffu, s[g][t], o);
                    if (r0 + t * RPL >= len) s[g][t] = -CUDART_INF_F;
                }
            // online softmax; the running maximum is uniform across the warp
            float w[GT][NI];
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float mx = s[g][0];
#pragma unroll
                for (int t = 1; t < NI; ++t) mx = fmaxf(mx, s[g][t]);
#pragma unroll
                for (int o = VEC; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float mn = fmaxf(m[g], mx);                 // finite: a pass holds >= 1 valid row
                const float corr = exp2f(m[g] - mn);              // first pass: exp2(-inf) = 0
                float ls = 0.f;
#pragma unroll
                for (int t = 0; t < NI; ++t) { w[g][t] = exp2f(s[g][t] - mn); ls += w[g][t]; }
                l[g] = l[g] * corr + ls;
                m[g] = mn;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][e] *= corr;
            }
#pragma unroll
            for (int t = 0; t < NI; ++t) {
                float vf[8];
                unpack8(vr[t], vf);
#pragma unroll
                for (int g = 0; g < GT; ++g)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[g][e] = fmaf(w[g][t], vf[e], acc[g][e]);
            }
        }
        // fold the row groups together, normalise, store
#pragma unroll
        for (int g = 0; g < GT; ++g) {
#pragma unroll
            for (int o = VEC; o < 32; o <<= 1) {
                l[g] += __shfl_xor_sync(0xffffffffu, l[g], o);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][e] += __shfl_xor_sync(0xffffffffu, acc[g][e], o);
            }
            if (rsub == 0) {
                const float inv = l[g] > 0.f ? 1.f / l[g] : 0.f;   // no valid key: zero row
                uint4 o4;
                o4.x = pack2(acc[g][0] * inv, acc[g][1] * inv);
                o4.y = pack2(acc[g][2] * inv, acc[g][3] * inv);
                o4.z = pack2(acc[g][4] * inv, acc[g][5] * inv);
                o4.w = pack2(acc[g][6] * inv, acc[g][7] * inv);
                *reinterpret_cast<uint4 *>(out_base + (size_t)(g0 + g) * DH) = o4;
            }
        }
    }
}

template <int DH, int RP, int GT>
cudaError_t launch(const AttnParams &p, cudaStream_t st, long long *launches) {
    const long long items = (long long)p.n_q * p.Hkv;
    // a plain launch: with thousands of CTAs in many waves an early start only parks CTAs on the SMs
    chunk_attn_kernel<DH, RP, GT><<<(unsigned)((items + CH_WARPS - 1) / CH_WARPS), CH_WARPS * 32, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

template <int DH, int RP>
cudaError_t pick_group(const AttnParams &p, cudaStream_t st, long long *launches) {
    const int G = p.Hq / p.Hkv;
    if (G % 4 == 0) return launch<DH, RP, 4>(p, st, launches);
    if (G % 2 == 0) return launch<DH, RP, 2>(p, st, launches);
    return launch<DH, RP, 1>(p, st, launches);
}

template <int DH>
cudaError_t pick_rows(const AttnParams &p, cudaStream_t st, long long *launches) {
    if (p.n_q == 0) return cudaSuccess;
    if (p.cap <= 8) return pick_group<DH, 8>(p, st, launches);
    if (p.cap <= 16) return pick_group<DH, 16>(p, st, launches);
    if (p.cap <= 24) return pick_group<DH, 24>(p, st, launches);
    return pick_group<DH, 32>(p, st, launches);          // longer buffers take several passes
}

}  // namespace

cudaError_t launch_chunk_attention(photon_ctx *, const AttnParams &p, cudaStream_t st,
                                   long long *launches) {
    return p.dh == 64 ? pick_rows<64>(p, st, launches) : pick_rows<128>(p, st, launches);
}
