// Chunk-local bounded attention of the local decoders (Eq. 6-7): every query
// attends the first len rows of its own chunk buffer only (R_l prefix rows plus
// the in-chunk rows written so far), so a problem is at most P + C <= 64 keys.
//
// HBM-bound streaming of many tiny problems.  A warp owns one (chunk, KV head):
// the valid K and V rows of that pair are one contiguous run of len * dh * 2
// bytes each; rows >= len are never touched.  A row is spread over dh/8 lanes;
// logits are reduced with warp shuffles, the softmax runs in the base-2 domain
// in fp32, and the G query heads of the group reuse the rows.  One launch, no
// workspace: the result is rounded once to bf16 and stored.
//
// Two kernels do that arithmetic and differ in how the rows arrive:
//  - chunk_attn_kernel: 128-bit loads into registers, all issued before the
//    first use (up to 2 * RP rows in flight per warp), one item per warp, many
//    small CTAs.  For small calls, and for buffers too large for the ring.
//  - chunk_attn_ring_kernel: one persistent CTA per SM; every consumer warp has
//    a private ring of RING_DEPTH items (K rows, V rows, queries) in shared
//    memory, which a producer warp keeps filled with bulk copies.  The next
//    item's rows are on their way while a warp computes, so the bytes in flight
//    per SM no longer drop while warps are busy with arithmetic: with registers
//    as the landing place a warp has nothing in flight for about half of its
//    time.  No consumer waits for another.
#include <math_constants.h>

#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

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

// The ring kernel's arithmetic.  DH: head size; RP: rows per pass (a pass covers rows [pass*RP, pass*RP + RP));
// GT: query heads evaluated together against the rows in registers.
//
// One item (query i, KV head kvh; numbered i * Hkv + kvh) against the first len rows of its buffer.  ldk(off) and
// ldv(off) give this lane the 16-byte vector that lies `off` vectors past its own place in the first rows (row lane / VEC, vector lane % VEC);
// ldq(off) likewise in the G query rows of the pair, from vector lane % VEC of the first.  `ok` says whether the row
// exists: a missing V row must come back as zeros (its weight is zero, but zero times whatever lies there need not
// be); a missing K row may come back as anything that can be read, its logit is replaced.
template <int DH, int RP, int GT, class LoadQ, class LoadK, class LoadV>
__device__ __forceinline__ void attend(const AttnParams &p, long long item, int len, int lane, LoadQ ldq, LoadK ldk, LoadV ldv) {
    constexpr int VEC = DH / 8;             // 16-byte vectors (= lanes) per row
    constexpr int RPL = 32 / VEC;           // rows covered by one warp-wide load
    constexpr int NI = RP / RPL;            // loads per lane per pass
    static_assert(RP % RPL == 0, "pass height must be a whole number of warp loads");
    const int G = p.Hq / p.Hkv;
    const int col = lane % VEC, rsub = lane / VEC;
    bf16 *out_base = p.out + (size_t)item * G * DH + col * 8;       // item = i * Hkv + kvh, and Hq = Hkv * G
    const int n_pass = (len + RP - 1) / RP;

    for (int g0 = 0; g0 < G; g0 += GT) {
        float qf[GT][8];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const uint4 qv = ldq((g0 + g) * VEC);
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
                kr[t] = ldk((pass * RP + t * RPL) * VEC, ok);
            }
#pragma unroll
            for (int t = 0; t < NI; ++t) {
                const bool ok = r0 + t * RPL < len;
                vr[t] = ldv((pass * RP + t * RPL) * VEC, ok);
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
            // Step by step over all logits: shuffles keep their order, a logit at a time would be one long chain, and
            // with few warps per SM nothing else fills the gaps.  (The register kernel, 16 warps per SM, is faster
            // with a logit at a time and fewer values live: measured both ways in both kernels.)
#pragma unroll
            for (int o = 1; o < VEC; o <<= 1)
#pragma unroll
                for (int g = 0; g < GT; ++g)
#pragma unroll
                    for (int t = 0; t < NI; ++t) s[g][t] += __shfl_xor_sync(0xffffffffu, s[g][t], o);
#pragma unroll
            for (int g = 0; g < GT; ++g)
#pragma unroll
                for (int t = 0; t < NI; ++t)
                    if (r0 + t * RPL >= len) s[g][t] = -CUDART_INF_F;
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

// A query whose unit index is out of range: flagged, and its output rows are zero (as are those of a query without keys).
template <int DH>
__device__ __forceinline__ void bad_index(const AttnParams &p, long long item, int lane, bool flag = true) {
    const int G = p.Hq / p.Hkv;
    if (flag && lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
    if (lane < DH / 8)
        for (int g = 0; g < G; ++g)
            *reinterpret_cast<uint4 *>(p.out + ((size_t)item * G + g) * DH + lane * 8) =
                make_uint4(0u, 0u, 0u, 0u);
}

// The register kernel: one item per warp, rows loaded straight into registers.  It has the arithmetic of `attend`
// written out once more (a logit at a time in the reduction, predicated loads, four heads at a time): sharing the
// function cost this kernel 15-20 % on small calls.
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

constexpr int RING_DEPTH = 2;               // items a consumer warp holds in shared memory: one in use, the next on its way
constexpr int RING_MAX_WARPS = 8;           // consumer warps per CTA
constexpr int RING_PRODUCERS = 4;           // producer warps on top of them
constexpr int RING_BATCH = 64;              // looked-up items a ring's table holds: the batch in use and the next one
constexpr int RING_BAR_BYTES = 2 * RING_MAX_WARPS * RING_DEPTH * 8;                     // full[w][d], then empty[w][d]
constexpr int RING_TABLE_BYTES = RING_MAX_WARPS * RING_BATCH * 8;                       // {block, len} per looked-up item

// half: bytes of one buffer's K (or V) rows for one KV head (cap * DH * 2).  A ring slot is K rows, V rows and the
// G query rows of the pair: the queries travel with the rows, or every item would start with a round trip to memory.
//
// Warps 0..W-1 consume: warp w takes items gw, gw + GW, ... (gw its number in the grid, GW the grid's consumer warps),
// looks unit and length up 32 items at a time, a batch ahead, and leaves them in its table for the producers.  The
// warps after them produce: one lane per ring, three bulk copies per item as soon as the slot is free.  Issuing those copies
// holds a warp for several hundred cycles per item (measured), which is why the consumers do not do it themselves.
template <int DH, int RP, int GT>
__global__ void __launch_bounds__((RING_MAX_WARPS + RING_PRODUCERS) * 32, 1)
chunk_attn_ring_kernel(const AttnParams p, int half) {
    constexpr int VEC = DH / 8;
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, W = (blockDim.x >> 5) - RING_PRODUCERS;
    const int G = p.Hq / p.Hkv;
    const uint32_t q_bytes = (uint32_t)G * DH * 2, slot_bytes = 2 * half + q_bytes;
    const uint32_t bars = ptx::smem_u32(smem);
    int2 *table = reinterpret_cast<int2 *>(smem + RING_BAR_BYTES);
    const uint32_t data = bars + RING_BAR_BYTES + RING_TABLE_BYTES;
    auto full = [&](int w, int d) { return bars + (w * RING_DEPTH + d) * 8; };
    auto empty = [&](int w, int d) { return bars + ((RING_MAX_WARPS + w) * RING_DEPTH + d) * 8; };
    if (threadIdx.x < W * RING_DEPTH) {
        ptx::mbar_init(full(0, threadIdx.x), 1);
        ptx::mbar_init(empty(0, threadIdx.x), 1);
        ptx::mbar_fence_init();
    }
    // Items go round the warps of the grid: neighbours in memory are fetched at about the same time.
    const int items = p.n_q * p.Hkv, GW = gridDim.x * W;
    auto count = [&](int gw) { return gw < items ? (items - gw + GW - 1) / GW : 0; };

    if (warp < W) {
        const int gw = blockIdx.x * W + warp, n_mine = count(gw);
        // block = u * Hkv + kvh, the item's run of cap rows in either cache; len = -1 for a unit out of range
        auto look = [&](int kb) {
            int2 b = make_int2(0, 0);
            if (kb + lane < n_mine) {
                const int n = gw + (kb + lane) * GW, i = n / p.Hkv;
                const int u = p.slot ? __ldcg(p.slot + i) : i;
                if (u < 0 || u >= p.n_units) b.y = -1;
                else b.x = u * p.Hkv + (n - i * p.Hkv), b.y = max(0, min(__ldcg(p.len + u), p.cap));
            }
            return b;
        };
        auto post = [&](int kb, int2 b) { table[warp * RING_BATCH + (kb + lane) % RING_BATCH] = b; };
        int kb = 0;
        int2 cur = look(0), nxt = look(32);
        post(0, cur);
        post(32, nxt);
        __syncthreads();                                 // barriers and the first two batches are there for the producer
        for (int k = 0; k < n_mine; ++k) {
            // The batch behind becomes the one in use and a new one is looked up; half a batch later, when the loads
            // have long returned, it goes into the table entries of the batch before, which the producer, never behind
            // this warp, has left.  The producer reads an entry only after this warp's arrival for an item of the
            // batch before it, RING_DEPTH items earlier: later than the store.
            if (k - kb == 32) {
                kb += 32;
                cur = nxt;
                nxt = look(kb + 32);
            }
            if (k - kb == 16 && kb > 0) post(kb + 32, nxt);
            const int len = __shfl_sync(0xffffffffu, cur.y, k - kb);
            const int n = gw + k * GW, d = k % RING_DEPTH;
            if (!ptx::mbar_wait(full(warp, d), (k / RING_DEPTH) & 1)) {
                if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
                return;
            }
            if (len > 0) {
                const uint32_t ka = data + (warp * RING_DEPTH + d) * slot_bytes + lane * 16, va = ka + half;
                const uint32_t qa = data + (warp * RING_DEPTH + d) * slot_bytes + 2 * half + (lane % VEC) * 16;
                attend<DH, RP, GT>(p, n, len, lane, [=](int off) { return ptx::lds128(qa + off * 16); },
                                   [=](int off, bool) { return ptx::lds128(ka + off * 16); },      // the slot holds cap rows
                                   [=](int off, bool ok) {
                                       const uint4 x = ptx::lds128(va + off * 16);
                                       return ok ? x : make_uint4(0u, 0u, 0u, 0u);
                                   });
            } else {
                bad_index<DH>(p, n, lane, len < 0);      // a query without keys: zero rows, no flag
            }
            __syncwarp();                                // every lane is done with the slot before it is filled again
            if (lane == 0) ptx::mbar_arrive(empty(warp, d));
        }
        return;
    }

    __syncthreads();
    // Producers: between them the warps' lanes serve one ring each, and none waits for another ring: every turn of the loop it looks whether its own
    // next slot is free, and fills it if so.  An item without rows still passes through both barriers (a plain arrival
    // on full), so that the two sides cannot get more than RING_DEPTH items apart.
    const int w = lane * RING_PRODUCERS + (warp - W), gw = blockIdx.x * W + w, n_mine = w < W ? count(gw) : 0;
    int r = 0;
    uint64_t last = ptx::globaltimer_ns();
    for (;;) {
        const bool more = r < n_mine;
        if (!__any_sync(0xffffffffu, more)) break;
        const int d = r % RING_DEPTH;
        const bool go = more && (r < RING_DEPTH || ptx::mbar_test_wait(empty(w, d), (r / RING_DEPTH - 1) & 1));
        if (go) {
            const int2 b = table[w * RING_BATCH + r % RING_BATCH];
            if (b.y > 0) {
                const size_t off = (size_t)b.x * p.cap * DH;
                const uint32_t bytes = (uint32_t)b.y * DH * 2, dst = data + (w * RING_DEPTH + d) * slot_bytes;
                ptx::mbar_arrive_expect_tx(full(w, d), 2 * bytes + q_bytes);
                ptx::bulk_load(dst, p.k + off, bytes, full(w, d));
                ptx::bulk_load(dst + half, p.v + off, bytes, full(w, d));
                ptx::bulk_load(dst + 2 * half, p.q + (size_t)(gw + r * GW) * G * DH, q_bytes, full(w, d));
            } else {
                ptx::mbar_arrive(full(w, d));
            }
            ++r;
        }
        if (__any_sync(0xffffffffu, go)) {
            last = ptx::globaltimer_ns();
        } else if (ptx::globaltimer_ns() - last > 2000000000ull) {     // nobody freed a slot for two seconds
            if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
            break;
        }
    }
}

template <int DH, int RP, int GT>
cudaError_t launch(photon_ctx *ctx, const AttnParams &p, cudaStream_t st, long long *launches) {
    const long long items = (long long)p.n_q * p.Hkv;
    // The ring where shared memory has room for at least four consumer warps and every warp of the grid gets some
    // rounds of items: below that the rings never fill and the small CTAs start faster.
    const int half = p.cap * DH * 2;
    const size_t slot = 2 * (size_t)half + (size_t)(p.Hq / p.Hkv) * DH * 2, fixed = RING_BAR_BYTES + RING_TABLE_BYTES;
    const int W = (int)std::min<size_t>(RING_MAX_WARPS, ((227 << 10) - fixed) / (RING_DEPTH * slot));
    if (W >= 4 && items < (1ll << 31) && (long long)p.n_units * p.Hkv < (1ll << 31) && items >= 8ll * ctx->sm_count * W) {
        const size_t smem = fixed + (size_t)W * RING_DEPTH * slot;
        constexpr int GR = GT > 2 ? 2 : GT;              // rows come from shared memory: a second turn over them is cheap, spills are not
        static size_t smem_set[kMaxDevices] = {};
        if (const cudaError_t e = ensure_dynamic_smem(chunk_attn_ring_kernel<DH, RP, GR>, smem, ctx->device, smem_set))
            return e;
        chunk_attn_ring_kernel<DH, RP, GR><<<ctx->sm_count, (W + RING_PRODUCERS) * 32, smem, st>>>(p, half);
        ++*launches;
        return cudaGetLastError();
    }
    // a plain launch: with thousands of CTAs in many waves an early start only parks CTAs on the SMs
    chunk_attn_kernel<DH, RP, GT><<<(unsigned)((items + CH_WARPS - 1) / CH_WARPS), CH_WARPS * 32, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

template <int DH, int RP>
cudaError_t pick_group(photon_ctx *ctx, const AttnParams &p, cudaStream_t st, long long *launches) {
    const int G = p.Hq / p.Hkv;
    if (G % 4 == 0) return launch<DH, RP, 4>(ctx, p, st, launches);
    if (G % 2 == 0) return launch<DH, RP, 2>(ctx, p, st, launches);
    return launch<DH, RP, 1>(ctx, p, st, launches);
}

template <int DH>
cudaError_t pick_rows(photon_ctx *ctx, const AttnParams &p, cudaStream_t st, long long *launches) {
    if (p.n_q == 0) return cudaSuccess;
    if (p.cap <= 8) return pick_group<DH, 8>(ctx, p, st, launches);
    if (p.cap <= 16) return pick_group<DH, 16>(ctx, p, st, launches);
    if (p.cap <= 24) return pick_group<DH, 24>(ctx, p, st, launches);
    return pick_group<DH, 32>(ctx, p, st, launches);          // longer buffers take several passes
}

}  // namespace

cudaError_t launch_chunk_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                                   long long *launches) {
    return p.dh == 64 ? pick_rows<64>(ctx, p, st, launches) : pick_rows<128>(ctx, p, st, launches);
}
