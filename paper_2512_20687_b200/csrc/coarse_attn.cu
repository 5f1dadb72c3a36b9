// Decode attention of the coarsest stream (attention half of STEP, Eq. 12) and
// of a token-level cache: one query position per unit over the valid rows of
// its own KV cache.  HBM-bound: every valid K and V row is streamed once.
//
// Work is cut into tiles of 64 keys of one (unit, KV head) stream.  The tiles
// of all streams, in stream order, form one sequence; a persistent grid (two
// CTAs per SM) gives every CTA an equal contiguous share of it, whatever the
// lengths of the individual caches, so there is one wave and no tail.  The
// split points are found on the device from len[] by a block-wide prefix sum;
// a split point that falls inside a short stream moves to the nearer end of it
// (a cut costs more than a few tiles of imbalance), long streams are cut.
//
// Inside a CTA one thread drives a ring of TMA loads (128-byte-swizzled boxes of
// 32 rows, so rows past the end of a cache are not fetched; the group's query
// rows ride along with the first tile of each stream), four warps consume the
// tiles, and a sixth warp finishes streams (everything that needs a round trip
// to global memory) while the consumers are already on the next stream.
// Each consumer warp takes 16 keys of every tile, evaluates S^T = K Q^T and
// O^T += V^T P^T with mma.sync tiles whose M side is the keys / head features
// and whose N side is the G <= 16 query heads of the group (so a 16-key block
// costs 2 * dh/16 MMAs whatever G is), and keeps an fp32 online softmax in the
// base-2 domain.  With G query rows per KV head the contraction has G flop per
// byte, far below the tensor ridge: the tensor pipe only has to keep pace with
// HBM, which is why this is not a tcgen05 kernel.
//
// A stream that lies inside one CTA is finished there.  A stream cut by a CTA
// boundary leaves one unnormalised partial (acc, m, l) per CTA in a small
// workspace; the CTA that arrives last on the stream's ticket (an atomic
// counter, no waiting) merges the partials in CTA order by log-sum-exp, so the
// result does not depend on arrival order.  Partials of a shared prefix, when
// present, were produced by an earlier launch and are folded in at the same
// point.
#include <math_constants.h>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int NW = 4;                      // consumer warps per CTA
constexpr int BN = 64;                     // keys per tile
constexpr int BOX = 32;                    // rows per TMA box of a tile's ragged end; whole tiles use boxes of BN rows
constexpr int THREADS = (NW + 2) * 32;     // + one producer warp + one finishing warp
constexpr int STAGES = 3;
constexpr int HALF_BYTES = BN * 128;       // 64 rows x 64 elements, swizzled
constexpr int BOX_BYTES = BOX * 128;
constexpr int CTAS_PER_SM = 2;
#ifndef COARSE_SNAP
#define COARSE_SNAP 8
#endif
constexpr int SNAP = COARSE_SNAP;          // streams of at most this many tiles are never cut
constexpr int NLEN = 768;                  // lengths of the first NLEN units are kept in shared memory

template <int DH>
struct Ring {
    static constexpr int HALVES = DH / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;     // K (or V) tile
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
};

__host__ __device__ inline int q_slot_bytes(int G, int dh) { return (G * dh * 2 + 127) / 128 * 128; }

template <int DH>
size_t smem_bytes(int G) {
    return size_t(STAGES) * (Ring<DH>::STAGE_BYTES + q_slot_bytes(G, DH) + 2 * DH * 2 /*a new K and V row*/) +
           size_t(NW) * G * (DH + 2) * sizeof(float) + 128 /*barriers*/ + 128 /*scalars*/ + NLEN * sizeof(int);
}

__device__ __forceinline__ int tiles_of(int len) { return (len + BN - 1) / BN; }

// Index arrays (lengths, page ids, prefix ids) are read through the L2 only: another kernel may have
// written them just before this one, and a line of them left in an SM's L1 by an earlier kernel is not
// refreshed by a dependent launch.
//
// A length is kept as it was read, clamped to [-1, cap] (-1: any negative value).  With the step's append
// folded into this kernel (p.k_new set) a unit with room grows by the one row the kernel itself installs:
// the keys it attends are those of the grown cache.
__device__ __forceinline__ int ld_len(const AttnParams &p, int u) { return max(-1, min(__ldcg(p.len + u), p.cap)); }
__device__ __forceinline__ bool appends(const AttnParams &p, int raw) { return p.k_new && raw >= 0 && raw < p.cap; }
__device__ __forceinline__ int eff_len(const AttnParams &p, int raw) { return appends(p, raw) ? raw + 1 : max(raw, 0); }

constexpr int LPT = NLEN / THREADS;        // lengths per thread when a batch fits the shared-memory copy
static_assert(NLEN % THREADS == 0, "a thread's units must fit its registers");

// The lengths of units [ub, ue), at most LPT of them, requested before any is used.
__device__ __forceinline__ void load_lengths(const AttnParams &p, int ub, int ue, int (&len)[LPT]) {
#pragma unroll
    for (int i = 0; i < LPT; ++i) len[i] = ub + i < ue ? __ldcg(p.len + ub + i) : 0;
#pragma unroll
    for (int i = 0; i < LPT; ++i) len[i] = max(-1, min(len[i], p.cap));
}

// A CTA's part of the tile sequence.
struct Share {
    long long T;             // tiles in the whole call
    int n_cta;               // CTAs that take part
    long long t0, t1;        // this CTA's tiles [t0, t1)
    int u0, rem;             // tile t0 is tile `rem` of the Hkv * nt tiles of unit u0
};

// Position in the sequence of tiles: tile j of the stream (unit u, KV head h).  The lengths of units
// [0, NLEN) sit in shared memory, read once per CTA; those of later units come from the L2.
struct Walker {
    int u, h, j, nt, len;
    bool app;                // the unit's last row is the one this kernel installs
    const int *slen;
    __device__ __forceinline__ void load(const AttnParams &p) {
        const int raw = u < NLEN ? slen[u] : ld_len(p, u);
        len = eff_len(p, raw);
        app = appends(p, raw);
        nt = tiles_of(len);
    }
    // false: the share does not start at a tile of unit u0 (the lengths changed under the kernel)
    __device__ __forceinline__ bool start(const AttnParams &p, const Share &sh, const int *lens) {
        slen = lens; u = sh.u0; h = 0; j = 0; nt = 0; len = 0; app = false;
        if (u < 0 || u >= p.n_units) return false;
        load(p);
        if (nt == 0 || sh.rem < 0 || sh.rem >= nt * p.Hkv) return false;
        h = sh.rem / nt; j = sh.rem % nt;
        return true;
    }
    __device__ __forceinline__ bool valid(const AttnParams &p) const { return u < p.n_units; }
    __device__ __forceinline__ void next(const AttnParams &p) {
        if (++j < nt) return;
        j = 0;
        if (++h < p.Hkv) return;
        h = 0;
        do {
            if (++u >= p.n_units) { u = p.n_units; nt = 0; len = 0; app = false; return; }
            load(p);
        } while (nt == 0);
    }
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

// Final value of one output element: own keys (acc, M, L in the base-2 domain,
// unnormalised) combined with the partials of the unit's shared prefix.
template <int DH>
__device__ __forceinline__ void emit(const AttnParams &p, int u, int hq, int d, float acc, float M, float L) {
    const size_t qh = (size_t)u * p.Hq + hq;
    if (p.splits_sh > 0) {
        const int s = __ldcg(p.sh_id + u);
        if (s >= p.n_shared) {                       // bad shared id voids the query
            if (d == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
            L = 0.f; acc = 0.f;
        } else if (s >= 0) {
            const float *pj = p.partials + qh * (DH + 2);
            const float lj = __ldcg(pj + DH + 1);
            if (lj > 0.f) {
                const float mj = __ldcg(pj + DH);
                const float Mn = fmaxf(M, mj);
                const float f0 = L > 0.f ? exp2f(M - Mn) : 0.f, f1 = exp2f(mj - Mn);
                acc = acc * f0 + __ldcg(pj + d) * f1;
                L = L * f0 + lj * f1;
                M = Mn;
            }
        }
    }
    p.out[qh * DH + d] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
    if (d == 0 && p.lse) p.lse[qh] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -CUDART_INF_F;
}

// The shared-prefix partial of one query head as the finishing warp holds it: fetched before the own keys
// of the stream are done, so that its latency hides behind the consumers' work.
template <int MAXV>
struct SharedPart {
    int sid;                 // prefix id of the unit (< 0: none)
    float l, m;
    float2 a[MAXV / 2];
};

template <int DH, int MAXV>
__device__ __forceinline__ void fetch_shared(const AttnParams &p, int u, int hq, int d0, SharedPart<MAXV> &sp) {
    sp.sid = -1;
    if (p.splits_sh <= 0) return;
    sp.sid = __ldcg(p.sh_id + u);
    if (sp.sid < 0 || sp.sid >= p.n_shared) return;
    const float *pj = p.partials + ((size_t)u * p.Hq + hq) * (DH + 2);
    sp.l = __ldcg(pj + DH + 1);
    sp.m = __ldcg(pj + DH);
#pragma unroll
    for (int i = 0; i < MAXV / 2; ++i) sp.a[i] = __ldcg(reinterpret_cast<const float2 *>(pj + d0) + i);
}

// The finishing warp holds, per lane, MAXV consecutive features [d0, d0 + MAXV) of one query head
// (acc unnormalised, M and L of that head).  Same combination as emit().
template <int DH, int MAXV>
__device__ __forceinline__ void emit_row(const AttnParams &p, int u, int hq, int d0, bool lead,
                                         float (&acc)[MAXV], float M, float L, const SharedPart<MAXV> &sp) {
    const size_t qh = (size_t)u * p.Hq + hq;
    if (p.splits_sh > 0) {
        if (sp.sid >= p.n_shared) {                  // bad shared id voids the query
            if (lead) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
            L = 0.f;
        } else if (sp.sid >= 0 && sp.l > 0.f) {
            const float Mn = fmaxf(M, sp.m);
            const float f0 = L > 0.f ? exp2f(M - Mn) : 0.f, f1 = exp2f(sp.m - Mn);
#pragma unroll
            for (int i = 0; i < MAXV / 2; ++i) {
                acc[2 * i] = acc[2 * i] * f0 + sp.a[i].x * f1;
                acc[2 * i + 1] = acc[2 * i + 1] * f0 + sp.a[i].y * f1;
            }
            L = L * f0 + sp.l * f1;
            M = Mn;
        }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    uint32_t *dst = reinterpret_cast<uint32_t *>(p.out + qh * DH + d0);
#pragma unroll
    for (int i = 0; i < MAXV / 2; ++i) dst[i] = pack_bf16(acc[2 * i] * inv, acc[2 * i + 1] * inv);
    if (lead && p.lse) p.lse[qh] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -CUDART_INF_F;
}

// One 16-key block of a tile for this warp.
//   kt, vt   shared-memory addresses of the K and V tiles (swizzled boxes)
//   kb       index of the 16-key block inside the tile;  valid: keys of it in range (1..16)
//   qb       Q^T fragments: [n-tile of 8 heads][16-wide slice of dh][2]
//   o        O^T accumulators: [n-tile][16-row slice of dh][4]
//   m, l     running maximum and (per-thread partial) sum for heads 2c, 2c+1 of each n-tile
template <int DH, int NT8>
__device__ __forceinline__ void process_block(uint32_t kt, uint32_t vt, int kb, int valid,
                                              const uint32_t (&qb)[NT8][DH / 16][2],
                                              float (&o)[NT8][DH / 16][4], float (&m)[NT8][2],
                                              float (&l)[NT8][2], float scale_log2, int lane) {
    const int g = lane >> 2, c = lane & 3;
    const int mi = lane >> 3, r8 = lane & 7;
    float s[NT8][2][4];
#pragma unroll
    for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[nt][a][e] = 0.f;

    // S^T = K Q^T : A fragments (keys x dh) straight from the swizzled K tile
    {
        const int row = kb * 16 + r8 + (mi & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            const int cfull = ks * 2 + (mi >> 1);                // 16-byte chunk along dh
            const uint32_t addr = kt + (cfull >> 3) * HALF_BYTES + row * 128 + (((cfull & 7) ^ (row & 7)) << 4);
            uint32_t a[4];
            ptx::ldmatrix_x4(a, addr);
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt) ptx::mma_bf16_16816(s[nt][ks & 1], a, qb[nt][ks][0], qb[nt][ks][1]);
        }
    }
    // online softmax over the keys (rows g and g+8 of the block), per head column
    uint32_t pb[NT8][2];
    bool rescale = false;
    float corr[NT8][2];
#pragma unroll
    for (int nt = 0; nt < NT8; ++nt) {
        float p_lo[2], p_hi[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float s_lo = (s[nt][0][j] + s[nt][1][j]) * scale_log2;            // key g
            float s_hi = (s[nt][0][2 + j] + s[nt][1][2 + j]) * scale_log2;    // key g + 8
            if (g >= valid) s_lo = -CUDART_INF_F;
            if (g + 8 >= valid) s_hi = -CUDART_INF_F;
            float mx = fmaxf(s_lo, s_hi);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float mn = fmaxf(m[nt][j], mx);                 // key 0 of a block is always in range
            corr[nt][j] = exp2f(m[nt][j] - mn);
            rescale |= (corr[nt][j] != 1.f);
            p_lo[j] = exp2f(s_lo - mn);
            p_hi[j] = exp2f(s_hi - mn);
            l[nt][j] = l[nt][j] * corr[nt][j] + (p_lo[j] + p_hi[j]);
            m[nt][j] = mn;
        }
        // P (keys x heads) -> P^T fragments (B operand: keys along k, head g of this thread)
        pb[nt][0] = ptx::movmatrix_trans(pack_bf16(p_lo[0], p_lo[1]));
        pb[nt][1] = ptx::movmatrix_trans(pack_bf16(p_hi[0], p_hi[1]));
    }
    // masks that clear V entries of keys past the end (they may hold anything)
    uint32_t vm0 = 0xFFFFFFFFu, vm1 = 0xFFFFFFFFu;
    if (valid < 16) {
        vm0 = (2 * c < valid ? 0x0000FFFFu : 0u) | (2 * c + 1 < valid ? 0xFFFF0000u : 0u);
        vm1 = (2 * c + 8 < valid ? 0x0000FFFFu : 0u) | (2 * c + 9 < valid ? 0xFFFF0000u : 0u);
    }
    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
            for (int mt = 0; mt < DH / 16; ++mt) {
                o[nt][mt][0] *= corr[nt][0]; o[nt][mt][1] *= corr[nt][1];
                o[nt][mt][2] *= corr[nt][0]; o[nt][mt][3] *= corr[nt][1];
            }
    }
    // O^T += V^T P^T : A fragments (dh x keys) through transposing loads of the V tile
    {
        const int row = kb * 16 + r8 + (mi >> 1) * 8;
#pragma unroll
        for (int mt = 0; mt < DH / 16; ++mt) {
            const int cfull = mt * 2 + (mi & 1);
            const uint32_t addr = vt + (cfull >> 3) * HALF_BYTES + row * 128 + (((cfull & 7) ^ (row & 7)) << 4);
            uint32_t a[4];
            ptx::ldmatrix_x4_trans(a, addr);
            a[0] &= vm0; a[1] &= vm0; a[2] &= vm1; a[3] &= vm1;
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt) ptx::mma_bf16_16816(o[nt][mt], a, pb[nt][0], pb[nt][1]);
        }
    }
}

// The even deal of the tile sequence over the grid, found by all threads of the CTA from len[]: every
// length is read once (and left in shared memory for units below NLEN), a block-wide prefix sum of tile
// counts follows, then the two boundaries of this CTA's share.  Boundary c is tile T*c/n_cta; where it
// falls inside a short stream (<= SNAP tiles) it moves to the nearer end of that stream (finishing a
// cut stream costs round trips to global memory, more than a few tiles of imbalance); long streams are
// cut.  sc: [0..5] warp sums, [8] u0, [9] rem, [12] t0, [14] t1.
__device__ __forceinline__ Share deal(const AttnParams &p, int *sc, int *slen, int cta) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto len_of = [&](int u) { return eff_len(p, u < NLEN ? slen[u] : ld_len(p, u)); };
    const int per = (p.n_units + THREADS - 1) / THREADS;
    const int ub = min(p.n_units, (int)threadIdx.x * per), ue = min(p.n_units, ub + per);
    int mine = 0;
    if (per <= LPT) {                                             // all loads in flight together
        int len[LPT];
        load_lengths(p, ub, ue, len);
#pragma unroll
        for (int i = 0; i < LPT; ++i)
            if (ub + i < ue) { slen[ub + i] = len[i]; mine += tiles_of(eff_len(p, len[i])); }
    } else {
        for (int u = ub; u < ue; ++u) {
            const int len = ld_len(p, u);
            if (u < NLEN) slen[u] = len;
            mine += tiles_of(eff_len(p, len));
        }
    }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sc[warp] = incl;
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < THREADS / 32; ++w) {
        if (w < warp) before += sc[w];
        all += sc[w];
    }
    Share sh;
    sh.T = (long long)all * p.Hkv;
    // every CTA that takes part owns at least one tile of the even deal, so the CTAs holding a cut stream
    // are consecutive
    sh.n_cta = (int)min((long long)gridDim.x, sh.T);
    {
        const long long lo = (long long)(before + incl - mine) * p.Hkv, hi = lo + (long long)mine * p.Hkv;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const int c = cta + which;
            if (cta >= sh.n_cta || c >= sh.n_cta) continue;
            // (64-bit division is a long instruction sequence on the way to the first load)
            const long long x = sh.T < (1 << 20) ? (long long)((unsigned)sh.T * (unsigned)c / (unsigned)sh.n_cta)
                                                 : sh.T * c / sh.n_cta;
            if (!(lo <= x && x < hi)) continue;
            long long pre = lo;
            for (int u = ub; u < ue; ++u) {
                const int nt = tiles_of(len_of(u));
                const long long k = (long long)nt * p.Hkv;
                if (x < pre + k) {                                // nt > 0 here
                    int rem = (int)(x - pre), uu = u;
                    const int j = rem % nt;
                    long long bx = x;
                    if (nt <= SNAP && j != 0) {
                        if (2 * j <= nt) { bx = x - j; rem -= j; }
                        else { bx = x + (nt - j); rem += nt - j; }
                    }
                    if (rem == nt * p.Hkv) {                      // moved to the start of the next unit that has keys
                        rem = 0;
                        do { ++uu; } while (uu < p.n_units && len_of(uu) == 0);
                    }
                    if (which == 0) { sc[8] = uu; sc[9] = rem; sc[12] = (int)bx; }
                    else sc[14] = (int)bx;
                    break;
                }
                pre += k;
            }
        }
    }
    __syncthreads();
    const bool in = cta < sh.n_cta;
    sh.t0 = in ? sc[12] : 0;
    sh.t1 = in ? (sc[14] >= 0 ? sc[14] : sh.T) : 0;
    sh.u0 = sc[8]; sh.rem = sc[9];
    return sh;
}

// Address of the first key row of tile w.j of the stream (w.u, w.h) as a row of the cache tensor
// (contiguous, or through the page table); -1 for a page id out of range.
__device__ __forceinline__ int tile_row(const AttnParams &p, const Walker &w) {
    if (!p.page_table) return (w.u * p.Hkv + w.h) * p.cap + w.j * BN;
    const int row = w.j * BN;
    const int id = __ldcg(p.page_table + (size_t)w.u * p.pages_per_unit + row / p.page_rows);
    if (id < 0 || id >= p.n_pages) return -1;
    return (id * p.Hkv + w.h) * p.page_rows + row % p.page_rows;
}

// GP: the group size G rounded up to a power of two (1 .. 16); it fixes how the finishing warp's lanes
// map to (query head, features) and how many n-tiles of 8 heads the MMAs span.
template <int DH, int GP>
__global__ void __launch_bounds__(THREADS, CTAS_PER_SM)
coarse_attn_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_k_end, const __grid_constant__ CUtensorMap tm_v_end) {
    using R = Ring<DH>;
    constexpr int NT8 = GP > 8 ? 2 : 1;
    extern __shared__ __align__(1024) uint8_t smem_raw[];      // the swizzled tiles want 1024-byte alignment
    const int G = p.Hq / p.Hkv;
    const int QB = q_slot_bytes(G, DH);
    constexpr int NB = 2 * DH * 2;                              // a new K row and a new V row
    const uint32_t base = ptx::smem_u32(smem_raw);
    uint8_t *gen = smem_raw;
    const uint32_t q_base = base + STAGES * R::STAGE_BYTES;
    const uint32_t n_base = q_base + STAGES * QB;               // per stage: the row a folded-in append installs
    float *red = reinterpret_cast<float *>(gen + STAGES * (R::STAGE_BYTES + QB + NB));  // [NW][G][DH + 2]
    uint8_t *tail = reinterpret_cast<uint8_t *>(red) + (size_t)NW * G * (DH + 2) * sizeof(float);
    const uint32_t bars = ptx::smem_u32(tail);                  // full[s] at +16s, empty[s] at +16s+8
    const uint32_t red_full = bars + 16 * STAGES, red_empty = red_full + 8;
    int *sc = reinterpret_cast<int *>(tail + 128);              // scalars of the deal, [11] dead,
    volatile int *dead = sc + 11;                               // [16..23] description of the stream in `red`
    volatile int *meta = sc + 16;
    int *slen = sc + 32;                                        // [NLEN] lengths of the first units

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    if (base & 1023u) {                                         // never expected: the ring would be misplaced
        if (threadIdx.x == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, NW);
        }
        ptx::mbar_init(red_full, NW);
        ptx::mbar_init(red_empty, 1);
        sc[8] = -1; sc[9] = 0; sc[11] = 0; sc[12] = 0; sc[14] = -1;
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_k); ptx::prefetch_tmap(&tm_v);
        ptx::prefetch_tmap(&tm_k_end); ptx::prefetch_tmap(&tm_v_end);
    }

    // ---- the deal, ahead of the kernel before this one.  The lengths as they read now may still change
    // (an append in flight), and no key or value is touched yet; after the dependency wait every length is
    // read again, and the deal stands if no unit's tile count differs (it depends on nothing else), so
    // that one trip to the L2 and one barrier are all that separates the wait from the first load.
    // Batches beyond NLEN units keep no copy to compare with and deal after the wait.
    const bool ahead = p.n_units <= NLEN;
    Share sh;
    Walker w;
    bool started = false;
    if (ahead) {
        sh = deal(p, sc, slen, cta);
        if (sh.t0 < sh.t1) started = w.start(p, sh, slen);
    }

    // One tile into stage it % STAGES: the walker's current tile, with the group's query rows if a stream starts
    // there and the row a folded-in append installs if the stream ends there.  whole_box: fetch a box of BN
    // rows whatever the length says (for loads that go out before the lengths are confirmed: a unit may have
    // grown inside its last tile since they were read; what lies past the end of a cache is never used).
    auto issue_tile = [&](int it, const Walker &tw, bool whole_box) {
        const int s = it % STAGES;
        // row of the tile's first key in the cache tensor; for a paged cache through the page table
        int y = tile_row(p, tw);
        if (y < 0) { atomicOr(p.status, PHOTON_DEV_BAD_INDEX); y = tw.h * (p.page_table ? p.page_rows : p.cap); }
        const uint32_t full = bars + 16 * s;
        const uint32_t kd = base + s * R::STAGE_BYTES, vd = kd + R::TILE_BYTES;
        const int rows = min(BN, tw.len - tw.j * BN);
        const bool first = (it == 0 || tw.j == 0);
        // a tile of more than BOX rows comes as one box of BN rows per 64 features, a shorter one as one box of BOX rows
        const bool tall = whole_box || rows > BOX;
        const bool grows = tw.app && tw.j == tw.nt - 1;        // the row this kernel installs lies in this tile
        ptx::mbar_arrive_expect_tx(full, R::HALVES * (tall ? HALF_BYTES : BOX_BYTES) * 2 + (first ? G * DH * 2 : 0) +
                                             (grows ? NB : 0));
#pragma unroll
        for (int hh = 0; hh < R::HALVES; ++hh) {
            ptx::tma_load_2d(kd + hh * HALF_BYTES, tall ? &tm_k : &tm_k_end, hh * 64, y, full);
            ptx::tma_load_2d(vd + hh * HALF_BYTES, tall ? &tm_v : &tm_v_end, hh * 64, y, full);
        }
        if (first)
            ptx::bulk_load(q_base + s * QB, p.q + ((size_t)tw.u * p.Hq + (size_t)tw.h * G) * DH, G * DH * 2, full);
        if (grows) {
            const size_t at = ((size_t)tw.u * p.Hkv + tw.h) * DH;                       // k_new, v_new: [n_units, Hkv, dh]
            ptx::bulk_load(n_base + s * NB, p.k_new + at, DH * 2, full);
            ptx::bulk_load(n_base + s * NB + DH * 2, p.v_new + at, DH * 2, full);
        }
    };

    ptx::grid_dep_wait();                   // lengths, caches and queries may come from the kernel before this one
    ptx::grid_dep_launch();                 // one wave of CTAs, all resident: the next kernel may line up behind them

    // The ring's first turn goes out at once, from the deal made ahead, while the lengths are read again: keys,
    // values and queries are final now, only the deal may turn out stale.  If it does (rare), these loads are
    // left to land, the ring's barriers are made anew and everything starts over from the deal.
    int n_early = 0;
    if (ahead && started && warp == NW && lane == 0) {
        const int n = (int)min((long long)STAGES, sh.t1 - sh.t0);
        for (; n_early < n && w.valid(p); ++n_early, w.next(p)) issue_tile(n_early, w, !p.k_new);
    }

    bool redo = !ahead;
    if (ahead) {
        const int per = (p.n_units + THREADS - 1) / THREADS;
        const int ub = min(p.n_units, (int)threadIdx.x * per), ue = min(p.n_units, ub + per);
        int diff = 0, len[LPT];
        load_lengths(p, ub, ue, len);
#pragma unroll
        for (int i = 0; i < LPT; ++i)
            if (ub + i < ue) {
                // (with the append folded in nothing else may change a length meanwhile: any difference counts,
                // and the loads that went out early were sized by the lengths themselves)
                diff |= p.k_new ? len[i] != slen[ub + i] : tiles_of(eff_len(p, len[i])) != tiles_of(eff_len(p, slen[ub + i]));
                slen[ub + i] = len[i];
            }
        redo = __syncthreads_or(diff);
    }
    if (redo) {
        if (ahead) {
            // what went out early belongs to a deal that no longer holds: let it land, then new barriers
            for (int b = 0; b < n_early; ++b)
                if (!ptx::mbar_wait(bars + 16 * b, 0)) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
            n_early = 0;
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int s = 0; s < STAGES; ++s) {
                    ptx::mbar_inval(bars + 16 * s);
                    ptx::mbar_init(bars + 16 * s, 1);
                }
                ptx::mbar_fence_init();
            }
        }
        if (threadIdx.x == 0) { sc[8] = -1; sc[9] = 0; sc[12] = 0; sc[14] = -1; }
        sh = deal(p, sc, slen, cta);
        started = sh.t0 < sh.t1 && w.start(p, sh, slen);
    } else if (started && w.valid(p)) {
        w.load(p);                          // same tile counts, but the unit may have grown within its last tile
    }
    const long long T = sh.T, t0 = sh.t0, t1 = sh.t1;
    const int n_cta = sh.n_cta;

    // ---- a folded-in append: from here on this CTA reads lengths from shared memory only (the host takes
    // this path for batches of at most NLEN units), and says so on a counter; the CTA that finds every
    // other one already there writes the grown lengths, and flags the units that had no room, with the
    // checks of the append kernel.  Its finishing warp does that while the first tiles are on their way.
    if (p.k_new && warp == NW + 1) {
        int last = 0;
        if (lane == 0) {
            last = (atomicAdd(p.readers, 1) == (int)gridDim.x - 1);
            if (last) *p.readers = 0;                          // zero again for the next call
        }
        if (__shfl_sync(0xffffffffu, last, 0)) {
            bool full = false;
            for (int u = lane; u < p.n_units; u += 32) {
                const int raw = slen[u];
                if (appends(p, raw)) p.len_w[u] = raw + 1;
                else full = true;
            }
            if (full) atomicOr(p.status, PHOTON_DEV_CAPACITY);
        }
    }

    // ---- units without own keys are visited by no tile: they are finished by whoever has time for it
    // (the whole CTA when it has no tiles, else the finishing warp before its first stream arrives)
    auto finish_empty_units = [&](int tid, int nthreads) {
        for (int u = cta; u < p.n_units; u += gridDim.x) {
            if (eff_len(p, u < NLEN ? slen[u] : ld_len(p, u)) != 0) continue;
            for (int idx = tid; idx < p.Hq * DH; idx += nthreads)
                emit<DH>(p, u, idx / DH, idx % DH, 0.f, -CUDART_INF_F, 0.f);
        }
    };
    if (t0 >= t1) {
        finish_empty_units(threadIdx.x, THREADS);
        return;
    }

    const int n_tiles = (int)(t1 - t0);
    if (!started) {
        // the deal and the lengths disagree: len[] changed while the kernel ran.  Nothing is loaded or written.
        if (threadIdx.x == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
        return;
    }

    if (warp == NW + 1) {
        // ======================= finishing warp =======================
        // lane -> (query head r of the group, features [d0, d0 + V))
        constexpr int MAXV = DH * GP / 32;
        constexpr int lpr = 32 / GP;                    // lanes per query head
        const int r = lane / lpr, d0 = (lane % lpr) * MAXV;
        const bool row_ok = r < G, lead = row_ok && (lane % lpr == 0);
        finish_empty_units(lane, 32);
        // it walks the streams of this CTA in the consumers' order, one step ahead of them
        Walker fw = w;
        for (int sidx = 0;; ++sidx) {
            SharedPart<MAXV> sp;
            sp.sid = -1;
            if (row_ok && fw.valid(p)) fetch_shared<DH, MAXV>(p, fw.u, fw.h * G + r, d0, sp);
            if (*dead || !ptx::mbar_wait(red_full, sidx & 1)) {
                if (!*dead) { *dead = 1; if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT); }
                break;
            }
            const int u = meta[0], h = meta[1], flags = meta[2], c_first = meta[3], c_last = meta[4];
            const bool whole = flags & 1, final_seg = flags & 2;
            if (flags & 4) break;                               // the consumers finish the CTA's last stream themselves
            if (u < 0 || u >= p.n_units || h < 0 || h >= p.Hkv || c_first < 0 || c_last >= (int)gridDim.x ||
                c_first > c_last) {
                // no such stream: the consumers ran past the last unit
                if (lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
                *dead = 1;
                break;
            }
            float acc[MAXV], M = -CUDART_INF_F, L = 0.f;
#pragma unroll
            for (int i = 0; i < MAXV; ++i) acc[i] = 0.f;
            if (row_ok) {
#pragma unroll
                for (int ww = 0; ww < NW; ++ww) {
                    const float *src = red + ((size_t)ww * G + r) * (DH + 2);
                    if (src[DH + 1] > 0.f) M = fmaxf(M, src[DH]);
                }
#pragma unroll
                for (int ww = 0; ww < NW; ++ww) {
                    const float *src = red + ((size_t)ww * G + r) * (DH + 2);
                    const float lw = src[DH + 1];
                    if (lw > 0.f) {
                        const float f = exp2f(src[DH] - M);
                        L += lw * f;
#pragma unroll
                        for (int i = 0; i < MAXV / 2; ++i) {
                            const float2 a = *reinterpret_cast<const float2 *>(src + d0 + 2 * i);
                            acc[2 * i] += a.x * f; acc[2 * i + 1] += a.y * f;
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(red_empty);          // consumers may reuse `red`
            if (whole) {
                if (row_ok) emit_row<DH, MAXV>(p, u, h * G + r, d0, lead, acc, M, L, sp);
            } else {
                // the stream is shared with neighbouring CTAs: leave a partial, whoever arrives last merges
                if (row_ok) {
                    float *dst = p.cta_partials + ((size_t)(2 * cta + (cta < c_last ? 1 : 0)) * G + r) * (DH + 2);
#pragma unroll
                    for (int i = 0; i < MAXV / 2; ++i)
                        *reinterpret_cast<float2 *>(dst + d0 + 2 * i) = make_float2(acc[2 * i], acc[2 * i + 1]);
                    if (lead) { dst[DH] = M; dst[DH + 1] = L; }
                }
                __threadfence();
                __syncwarp();
                int last = 0;
                if (lane == 0) {
                    int *ticket = p.tickets + (size_t)u * p.Hkv + h;
                    last = (atomicAdd(ticket, 1) == c_last - c_first);
                    if (last) *ticket = 0;                       // zero again for the next call
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    __threadfence();
                    if (row_ok) {
                        M = -CUDART_INF_F; L = 0.f;
#pragma unroll
                        for (int i = 0; i < MAXV; ++i) acc[i] = 0.f;
                        // PB partials per trip: all their loads are in flight together
                        constexpr int PB = MAXV <= 16 ? 4 : 2;
                        for (int cc = c_first; cc <= c_last; cc += PB) {
                            float mj[PB], lj[PB];
                            float2 a[PB][MAXV / 2];
#pragma unroll
                            for (int t = 0; t < PB; ++t) {
                                const int c2 = min(cc + t, c_last);
                                const float *src = p.cta_partials +
                                                   ((size_t)(2 * c2 + (c2 < c_last ? 1 : 0)) * G + r) * (DH + 2);
                                lj[t] = __ldcg(src + DH + 1); mj[t] = __ldcg(src + DH);
#pragma unroll
                                for (int i = 0; i < MAXV / 2; ++i)
                                    a[t][i] = __ldcg(reinterpret_cast<const float2 *>(src + d0) + i);
                            }
#pragma unroll
                            for (int t = 0; t < PB; ++t) {
                                if (cc + t > c_last || !(lj[t] > 0.f)) continue;
                                const float Mn = fmaxf(M, mj[t]);
                                const float f0 = exp2f(M - Mn), f1 = exp2f(mj[t] - Mn);   // M = -inf at first: f0 = 0
#pragma unroll
                                for (int i = 0; i < MAXV / 2; ++i) {
                                    acc[2 * i] = acc[2 * i] * f0 + a[t][i].x * f1;
                                    acc[2 * i + 1] = acc[2 * i + 1] * f0 + a[t][i].y * f1;
                                }
                                L = L * f0 + lj[t] * f1;
                                M = Mn;
                            }
                        }
                        emit_row<DH, MAXV>(p, u, h * G + r, d0, lead, acc, M, L, sp);
                    }
                }
            }
            if (final_seg) break;
            fw.j = fw.nt - 1;                                   // on to the next stream
            fw.next(p);
        }
        return;
    }

    if (warp == NW) {
        // ======================= producer: one thread feeds the ring =======================
        if (lane == 0) {
            int it = n_early;                                    // this thread's walker stands behind the tiles that went out early
            for (; it < n_tiles; ++it, w.next(p)) {
                const int s = it % STAGES;
                if (*dead) break;
                if (!w.valid(p)) {                               // ran past the last unit: len[] changed under the kernel
                    *dead = 1; atomicOr(p.status, PHOTON_DEV_BAD_INDEX); break;
                }
                // the ring starts empty: only from its second turn on is there a stage to wait for
                if (it >= STAGES && !ptx::mbar_wait(bars + 16 * s + 8, ((it / STAGES) & 1) ^ 1)) {
                    *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT); break;
                }
                issue_tile(it, w, false);
            }
            if (*dead) {
                // loads already issued still land in this CTA's shared memory: give them time to finish
                for (int b = max(0, it - STAGES); b < it; ++b) ptx::mbar_wait(bars + 16 * (b % STAGES), (b / STAGES) & 1);
            }
        }
        return;
    }

    // ======================= consumers =======================
    const int g = lane >> 2, c = lane & 3;
    uint32_t qb[NT8][DH / 16][2];
    float o[NT8][DH / 16][4];
    float m[NT8][2], l[NT8][2];
    int seg_j0 = 0;                                    // first tile of the stream this CTA saw
    long long seg_t = 0;                               // position of the stream's tile 0 in the sequence
    int sidx = 0;                                      // streams handed to the finishing warp so far

    for (int it = 0; it < n_tiles; ++it) {
        const int s = it % STAGES;
        if (!*dead && !ptx::mbar_wait(bars + 16 * s, (it / STAGES) & 1)) {
            *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT);
        }
        if (it == 0 || w.j == 0) {
            // a new stream starts: fetch the group's query rows, clear the running state
            seg_j0 = w.j;
            seg_t = t0 + it - w.j;
            const uint32_t qs = q_base + s * QB;
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    const int head = nt * 8 + g;
                    uint32_t v0 = 0u, v1 = 0u;
                    if (head < G) {
                        v0 = ptx::lds32(qs + (head * DH + ks * 16 + 2 * c) * 2);
                        v1 = ptx::lds32(qs + (head * DH + ks * 16 + 8 + 2 * c) * 2);
                    }
                    qb[nt][ks][0] = v0; qb[nt][ks][1] = v1;
                }
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt) {
                m[nt][0] = m[nt][1] = -CUDART_INF_F;
                l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
                for (int mt = 0; mt < DH / 16; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[nt][mt][e] = 0.f;
            }
        }
        if (w.app && w.j == w.nt - 1 && !*dead) {
            // The append of the step, folded in: the unit's newest row is not in the cache yet.  The warp whose
            // keys include it copies it from where it landed beside the tile into the tile (at its swizzled
            // place) and into the cache; no other warp reads those 16 keys.  Lane -> one 16-byte piece of K or V.
            const int r = w.len - 1 - w.j * BN;
            if ((r >> 4) == warp) {
                constexpr int PIECES = DH / 8;
                if (lane < 2 * PIECES) {
                    const bool is_v = lane >= PIECES;
                    const int cf = lane % PIECES;
                    const uint4 piece = ptx::lds128(n_base + s * NB + lane * 16);
                    const uint32_t tile = base + s * R::STAGE_BYTES + (is_v ? R::TILE_BYTES : 0);
                    ptx::sts128(tile + (cf >> 3) * HALF_BYTES + r * 128 + (((cf & 7) ^ (r & 7)) << 4), piece);
                    const size_t row = ((size_t)w.u * p.Hkv + w.h) * p.cap + (w.len - 1);
                    *reinterpret_cast<uint4 *>((is_v ? p.v_w : p.k_w) + row * DH + cf * 8) = piece;
                }
                __syncwarp();
            }
        }
        {
            const uint32_t kt = base + s * R::STAGE_BYTES, vt = kt + R::TILE_BYTES;
            const int v = min(BN, w.len - w.j * BN) - 16 * warp;
            if (v > 0 && !*dead) process_block<DH, NT8>(kt, vt, warp, min(v, 16), qb, o, m, l, p.scale_log2, lane);
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bars + 16 * s + 8);

        const bool stream_end = (w.j == w.nt - 1);
        if (stream_end || it == n_tiles - 1) {
            // ---- this warp's state goes into `red`: for the finishing warp, or, when this is the CTA's last
            // stream and it is complete, for the consumer warps themselves (each takes a quarter of the rows:
            // nothing else is left to do, and four warps are through sooner than one)
            const bool whole = stream_end && seg_j0 == 0, final_seg = (it == n_tiles - 1);
            const bool direct = whole && final_seg && p.splits_sh == 0;
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    l[nt][j] += __shfl_xor_sync(0xffffffffu, l[nt][j], 4);
                    l[nt][j] += __shfl_xor_sync(0xffffffffu, l[nt][j], 8);
                    l[nt][j] += __shfl_xor_sync(0xffffffffu, l[nt][j], 16);
                }
            if (!*dead && !ptx::mbar_wait(red_empty, (sidx & 1) ^ 1)) {
                *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT);
            }
#pragma unroll
            for (int nt = 0; nt < NT8; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int head = nt * 8 + 2 * c + j;
                    if (head < G) {
                        float *dst = red + ((size_t)warp * G + head) * (DH + 2);
#pragma unroll
                        for (int mt = 0; mt < DH / 16; ++mt) {
                            dst[mt * 16 + g] = o[nt][mt][j];
                            dst[mt * 16 + 8 + g] = o[nt][mt][2 + j];
                        }
                        if (g == 0) { dst[DH] = m[nt][j]; dst[DH + 1] = l[nt][j]; }
                    }
                }
            if (warp == 0 && lane == 0) {
                meta[0] = w.u; meta[1] = w.h;
                meta[2] = (whole ? 1 : 0) | (final_seg ? 2 : 0) | (direct ? 4 : 0);
                meta[3] = meta[4] = cta;
                if (!whole) {
                    // CTAs that hold a piece of this stream: first and last
                    const long long te = seg_t + w.nt;
                    meta[3] = (int)(((seg_t + 1) * n_cta - 1) / T);
                    meta[4] = (int)((te * n_cta - 1) / T);
                }
            }
            if (direct) ptx::named_bar_sync(1, NW * 32);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(red_full);
            ++sidx;
            if (direct && !*dead) {
                // thread -> four consecutive features of one query head; same arithmetic as the finishing warp's
                for (int e = (warp * 32 + lane) * 4; e < G * DH; e += NW * 32 * 4) {
                    const int r = e / DH, d0 = e % DH;
                    float acc[4] = {0.f, 0.f, 0.f, 0.f}, M = -CUDART_INF_F, L = 0.f;
#pragma unroll
                    for (int ww = 0; ww < NW; ++ww) {
                        const float *src = red + ((size_t)ww * G + r) * (DH + 2);
                        if (src[DH + 1] > 0.f) M = fmaxf(M, src[DH]);
                    }
#pragma unroll
                    for (int ww = 0; ww < NW; ++ww) {
                        const float *src = red + ((size_t)ww * G + r) * (DH + 2);
                        const float lw = src[DH + 1];
                        if (lw > 0.f) {
                            const float f = exp2f(src[DH] - M);
                            L += lw * f;
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const float2 a = *reinterpret_cast<const float2 *>(src + d0 + 2 * i);
                                acc[2 * i] += a.x * f; acc[2 * i + 1] += a.y * f;
                            }
                        }
                    }
                    const float inv = L > 0.f ? 1.f / L : 0.f;
                    const size_t qh = (size_t)w.u * p.Hq + (size_t)w.h * G + r;
                    *reinterpret_cast<uint2 *>(p.out + qh * DH + d0) =
                        make_uint2(pack_bf16(acc[0] * inv, acc[1] * inv), pack_bf16(acc[2] * inv, acc[3] * inv));
                    if (d0 == 0 && p.lse) p.lse[qh] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -CUDART_INF_F;
                }
            }
        }
        w.next(p);
    }
}

template <int DH, int GP>
cudaError_t run(photon_ctx *ctx, AttnParams p, cudaStream_t st, long long *launches) {
    const int G = p.Hq / p.Hkv;
    const size_t smem = smem_bytes<DH>(G);
    static size_t smem_set[kMaxDevices] = {};
    if (const cudaError_t e = ensure_dynamic_smem(coarse_attn_kernel<DH, GP>, smem, ctx->device, smem_set)) return e;
    const CUtensorMap *t;
    CUtensorMap mk, mv, mk_end, mv_end;
    const uint64_t pool_rows = p.page_table ? (uint64_t)p.n_pages * p.Hkv * p.page_rows : (uint64_t)p.n_units * p.Hkv * p.cap;
    if (!(t = ctx->tmaps.get(p.k, pool_rows, DH, BN))) return cudaErrorInvalidValue;
    mk = *t;
    if (!(t = ctx->tmaps.get(p.v, pool_rows, DH, BN))) return cudaErrorInvalidValue;
    mv = *t;
    if (!(t = ctx->tmaps.get(p.k, pool_rows, DH, BOX))) return cudaErrorInvalidValue;
    mk_end = *t;
    if (!(t = ctx->tmaps.get(p.v, pool_rows, DH, BOX))) return cudaErrorInvalidValue;
    mv_end = *t;
    const int max_len = p.k_new ? std::min(p.max_len + 1, p.cap) : p.max_len;     // a folded-in append grows every unit by a row
    const long long t_max = (long long)p.n_units * p.Hkv * ((max_len + BN - 1) / BN);
    const long long cap = ctx->attn_ctas > 0 ? ctx->attn_ctas : coarse_attn_grid(ctx->max_ctas, (long long)p.n_units * p.Hkv);
    const int grid = (int)std::max<long long>(1, std::min<long long>(t_max, cap));
    const cudaError_t e = launch_dependent(coarse_attn_kernel<DH, GP>, dim3(grid), dim3(THREADS), smem, st, 0, p, mk, mv, mk_end, mv_end);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

int coarse_attn_ctas_per_sm() { return CTAS_PER_SM; }
int coarse_attn_fold_limit() { return NLEN; }

// The grid when the caller sets none.  Not every CTA slot of the device is taken: the kernel is bound by
// HBM well below that, and a slot left free lets a CTA of the next kernel in the stream start, and get
// through its set-up, while this one still runs (measured on caches of 64 to 256 MiB: 7/8 of the slots is 1 to 4 %
// faster than all of them).  Below that bound the grid is a multiple or a near-divisor of the number of
// (unit, KV head) streams, so that in a batch of equal lengths every stream falls to the same whole
// number of CTAs, or every CTA to the same whole number of streams, and the cuts of the even deal line
// up with the streams' ends; with ragged lengths the deal is even whatever the grid.
int coarse_attn_grid(int resident_ctas, long long n_streams) {
    const int top = std::max(1, resident_ctas * 7 / 8);
    if (n_streams <= 0) return 1;
    if (n_streams <= top) return (int)(n_streams * (top / n_streams));
    // more streams than CTAs: the grid within the upper quarter that wastes the fewest stream slots
    int best = top;
    long long best_waste = -1;
    for (int g = top; g >= top - top / 4; --g) {
        const long long waste = (n_streams + g - 1) / g * g - n_streams;
        if (best_waste < 0 || waste < best_waste) { best = g; best_waste = waste; }
        if (waste == 0) break;
    }
    return best;
}

cudaError_t launch_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st, long long *launches) {
    if (p.n_q == 0) return cudaSuccess;
    if (p.splits_sh > 0) {
        // Short own caches (at most one TMA box of rows per unit, by the caller's bound) ride along in the
        // shared-prefix kernel as extra key tiles, and that kernel writes the result: one launch instead of two.
        AttnParams ps = p;
        ps.own_rows = (!p.page_table && !p.k_new && p.max_len <= shared_prefix_own_rows()) ? shared_prefix_own_rows() : 0;
        const cudaError_t e = launch_shared_prefix_attention(ctx, ps, st, launches);
        if (e != cudaSuccess || ps.own_rows) return e;
    }
    const int G = p.Hq / p.Hkv;
    int gp = 1;
    while (gp < G) gp <<= 1;
#define PHOTON_COARSE_CASE(D, GPV) if (p.dh == D && gp == GPV) return run<D, GPV>(ctx, p, st, launches);
    PHOTON_COARSE_CASE(128, 1) PHOTON_COARSE_CASE(128, 2) PHOTON_COARSE_CASE(128, 4) PHOTON_COARSE_CASE(128, 8)
    PHOTON_COARSE_CASE(128, 16)
    PHOTON_COARSE_CASE(64, 1) PHOTON_COARSE_CASE(64, 2) PHOTON_COARSE_CASE(64, 4) PHOTON_COARSE_CASE(64, 8)
    PHOTON_COARSE_CASE(64, 16)
#undef PHOTON_COARSE_CASE
    return cudaErrorInvalidValue;
}
