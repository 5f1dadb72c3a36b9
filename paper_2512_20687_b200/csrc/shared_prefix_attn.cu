// Shared-prefix phase of the coarse decode attention (Section 1: long-context,
// multi-query serving): many units (query branches) attend the same stored
// prefix.  With hundreds of query rows per KV head this is a dense contraction,
// so it runs on the 5th-generation tensor cores, and the prefix is read once per
// group of 128 query rows instead of once per unit.
//
// CTA = (tile of 128 query rows = 128/G units x G heads, KV head, key range of
// the prefix).  Per 128-key tile:  S = Q K^T (tcgen05.mma, both operands
// K-major from 128B-swizzled shared memory, S in TMEM);  eight softmax warps read
// S with tcgen05.ld (two threads share a query row, 64 keys each, and exchange
// their maxima through shared memory), turn it into probabilities in the base-2
// domain and store them as bf16 into a swizzled shared-memory tile P;  O += P V (tcgen05.mma, V as the N-major operand
// straight from its TMA tile, O in TMEM across all tiles).  S is double
// buffered, so the tensor pipe computes the next S while the warps work on this
// one.  The reference maximum of a row is only raised when a tile exceeds it by
// more than 2^8; then the row's O (and its running sum) is rescaled in TMEM
// (tcgen05.ld / tcgen05.st).  Otherwise P simply carries factors up to 2^8.
//
// The key ranges of one row tile (1, 2, 4 or 8 of them) are the CTAs of one
// thread-block cluster: at the end every CTA sends its rows to the CTA that owns
// them (bulk copies into the peer's shared memory), each CTA merges the rows it owns
// by log-sum-exp, and the cluster leaves ONE unnormalised partial (acc, m, l) per query head at
// partials[query head]; the kernel that streams the units' own keys folds it
// into its result.  Units of a tile that
// name different prefixes are served in one pass per distinct prefix; a row
// takes part only in the pass of its own prefix.
#include <math_constants.h>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int BM = 128;                    // query rows per CTA (UMMA M; one TMEM lane each)
constexpr int BN = 128;                    // keys per tile
constexpr int KV_STAGES = 2;
constexpr int SW = 16;                     // softmax warps: warp w works on TMEM lanes 32*(w%4).., keys CH*(w/4)..
constexpr int KP = SW / 4;                 // threads that share a query row, each on CH keys of a tile
constexpr int CH = BN / KP;
constexpr int SP_THREADS = (SW + 3) * 32;  // + K loader + MMA warp and TMEM owner + V loader
constexpr float RESCALE_GAP = 8.f;         // log2 of the largest factor P may carry
constexpr int OWN = 32;                    // own rows per unit that can ride along (one TMA box); 128 / OWN units per key tile
constexpr int LIST = BM + BM / (BN / OWN); // entries of a CTA's tile list: distinct prefixes, then tiles of own keys

template <int DH>
struct SpTile {
    static constexpr int HALVES = DH / 64;
    static constexpr int Q_BYTES = HALVES * BM * 128;
    static constexpr int P_BYTES = (BN / 64) * BM * 128;
    static constexpr int KV_BYTES = HALVES * BN * 128;          // K (or V) tile
    static constexpr int OFF_P = Q_BYTES;
    static constexpr int OFF_K = OFF_P + P_BYTES;
    static constexpr int OFF_V = OFF_K + KV_STAGES * KV_BYTES;
    static constexpr int OFF_TAIL = OFF_V + KV_STAGES * KV_BYTES;
    // after the tiles: barriers (256), scalars (64), prefix ids (BM ints), maxima exchange (2 x 2 x BM floats),
    // sums exchange (2 x BM floats), the tile's distinct prefix ids with this CTA's key range of each (3 x BM ints),
    // lengths of the first 32 prefixes (32 ints)
    static constexpr int SMEM = OFF_TAIL + 1024 /*alignment slack*/ + 256 + 64 + BM * 4 + 2 * KP * BM * 4 + KP * BM * 4 +
                                3 * LIST * 4 + 32 * 4 + BM * 4 /*own lengths per unit of the tile*/;
    static constexpr int TMEM_COLS = 512;                       // S0, S1 (128 each), O (DH): next power of two
    static constexpr int COL_O = 2 * BN;
};

__device__ __forceinline__ void part_range(int L, int n_splits, int p, int &r0, int &r1) {
    const int per = ((L + n_splits - 1) / n_splits + BN - 1) / BN * BN;      // whole tiles per range
    r0 = min(L, p * per);
    r1 = min(L, r0 + per);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

template <int DH>
__global__ void __launch_bounds__(SP_THREADS, 1)
shared_prefix_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_ks, const __grid_constant__ CUtensorMap tm_vs,
                     const __grid_constant__ CUtensorMap tm_ko, const __grid_constant__ CUtensorMap tm_vo) {
    using T = SpTile<DH>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t sQ = base, sP = base + T::OFF_P, sK = base + T::OFF_K, sV = base + T::OFF_V;
    const uint32_t bars = base + T::OFF_TAIL;
    // barriers (8 bytes each)
    const uint32_t k_full = bars, v_full = bars + 16, k_empty = bars + 32, v_empty = bars + 112;   // [KV_STAGES]
    const uint32_t s_ready = bars + 48, s_free = bars + 64;                      // [2]
    const uint32_t p_ready = bars + 80, p_free = bars + 88, recv_bar = bars + 96;
    int *sc = reinterpret_cast<int *>(gen + T::OFF_TAIL + 256);                  // [0] tmem base, [1..2] rescale flags
    int *sid = sc + 16;                                                          // [BM] prefix id per query row's unit
    float *xch_m = reinterpret_cast<float *>(sid + BM);                          // [2 tiles in flight][KP key parts][BM]
    float *xch_l = xch_m + 2 * KP * BM;                                          // [KP key parts][BM]
    int *ids = reinterpret_cast<int *>(xch_l + KP * BM);                          // [BM] distinct prefix ids of the tile, ascending
    int *rng0 = ids + LIST, *rng1 = rng0 + LIST;                                 // this CTA's key range of each
    int *shl = rng1 + LIST;                                                      // [32] lengths of prefixes 0..31
    int *ulen = shl + 32;                                                        // [BM] own length of unit unit0 + i (0: none)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.Hq / p.Hkv;
    const int upt = BM / G;                                                      // units per tile
    const int part = blockIdx.x % p.splits_sh;                                   // = rank in the cluster
    const int h = (blockIdx.x / p.splits_sh) % p.Hkv;
    const int unit0 = (blockIdx.x / (p.splits_sh * p.Hkv)) * upt;
    constexpr int RS = DH + 4;                                                   // floats per staged row (16-byte aligned)
    const int C = p.splits_sh, rows_per = BM / C;

    if (threadIdx.x == 0) {
        for (int s = 0; s < KV_STAGES; ++s) {
            ptx::mbar_init(k_full + 8 * s, 1);
            ptx::mbar_init(v_full + 8 * s, 1);
            ptx::mbar_init(k_empty + 8 * s, 1);
            ptx::mbar_init(v_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(s_ready + 8 * b, 1);
            ptx::mbar_init(s_free + 8 * b, SW);
        }
        ptx::mbar_init(p_ready, SW);
        ptx::mbar_init(p_free, 1);
        ptx::mbar_init(recv_bar, 1);
        sc[1] = 0; sc[2] = 0;
        ptx::mbar_fence_init();
        // the rows this CTA owns arrive from the other CTAs of its cluster at the very end
        if (C > 1) ptx::mbar_arrive_expect_tx(recv_bar, (C - 1) * rows_per * RS * 4);
        else ptx::mbar_arrive(recv_bar);
        ptx::prefetch_tmap(&tm_ks); ptx::prefetch_tmap(&tm_vs);
    }
    ptx::grid_dep_wait();                      // queries may come from the kernel before this one
    ptx::grid_dep_launch();                    // one wave: the kernel for the units' own keys may line up
    // The Q tile goes to shared memory K-major with the 128-byte swizzle TMA would use.  Every warp but the two
    // loaders takes part; all of a thread's loads are requested here, before anything else, and stored once the
    // tile list below is done: one round trip to memory, under the one the ids make.
    constexpr int NQT = SP_THREADS - 64;
    constexpr int QV = (BM * (DH / 8) + NQT - 1) / NQT;
    const int tq = threadIdx.x < SW * 32 ? threadIdx.x : threadIdx.x - 32;
    uint4 qv[QV];
    if (warp != SW && warp != SW + 2) {
#pragma unroll
        for (int t = 0; t < QV; ++t) {
            const int idx = tq + t * NQT;
            const int r = idx / (DH / 8), ch = idx % (DH / 8);                   // 16-byte chunk ch of row r
            const int i = unit0 + r / G;
            qv[t] = make_uint4(0u, 0u, 0u, 0u);
            if (idx < BM * (DH / 8) && r < upt * G && i < p.n_q)
                qv[t] = __ldcg(reinterpret_cast<const uint4 *>(p.q + ((size_t)i * p.Hq + (size_t)h * G + r % G) * DH + ch * 8));
        }
    }
    // prefix id of every row's unit (>= 0 valid, -1 none or past the batch, -2 no such prefix); row r = (unit - unit0)
    // * G + g.  With the units' own keys riding along (p.own_rows = OWN: every unit holds at most OWN rows), the
    // own length of unit unit0 + r as well.  Both loads are requested before either is used.
    if (threadIdx.x < BM) {
        const int r = threadIdx.x, i = unit0 + r / G, u = unit0 + r;
        const bool has_row = r < upt * G && i < p.n_q, has_unit = p.own_rows && r < upt && u < p.n_q;
        int s = has_row ? __ldcg(p.sh_id + i) : -1;
        int n = has_unit ? __ldcg(p.len + u) : 0;
        if (s >= p.n_shared) s = -2;           // a prefix that does not exist voids the query
        else if (s < 0) s = -1;
        n = max(0, min(n, p.cap));
        if (n > OWN) { n = OWN; atomicOr(p.status, PHOTON_DEV_BAD_INDEX); }   // beyond what the caller's max_len promised
        sid[r] = s;
        ulen[r] = n;
    }
    // (the lengths of the first prefixes travel with the ids: one trip to the L2 for both)
    if (threadIdx.x >= SP_THREADS - 32) {
        const int i = threadIdx.x - (SP_THREADS - 32);
        shl[i] = i < p.n_shared ? max(0, min(__ldcg(p.sh_len + i), p.cap_sh)) : 0;
    }
    __syncthreads();
    // The list every role walks: the distinct prefix ids of the tile's units in ascending order, each with
    // this CTA's key range of that prefix.  One warp finds it (a minimum over the lanes per distinct id).
    if (warp == 0) {
        int n = 0, last = -1;
        for (;;) {
            int cand = 0x7FFFFFFF;
            for (int r = lane * G; r < BM; r += 32 * G) {
                const int s = sid[r];
                if (s > last && s < cand) cand = s;
            }
            const int cur = __reduce_min_sync(0xffffffffu, cand);
            if (cur == 0x7FFFFFFF) break;
            if (lane == 0) {
                const int L = cur < 32 ? shl[cur] : max(0, min(__ldcg(p.sh_len + cur), p.cap_sh));
                int r0, r1;
                part_range(L, p.splits_sh, part, r0, r1);
                ids[n] = cur; rng0[n] = r0; rng1[n] = r1;
            }
            ++n;
            last = cur;
        }
        // then the tiles of own keys: tile t holds the rows of units 4t .. 4t + 3 of this row tile; the key ranges of
        // the cluster take them in turn.  An entry with a negative id -1 - t stands for own tile t.
        if (p.own_rows) {
            const int n_own = (upt + BN / OWN - 1) / (BN / OWN);
            for (int t = part; t < n_own; t += p.splits_sh, ++n)
                if (lane == 0) { ids[n] = -1 - t; rng0[n] = 0; rng1[n] = BN; }
        }
        if (lane == 0) sc[3] = n;
    }
    __syncthreads();                           // barriers, ids and key ranges are ready: the TMA warps start loading at once
    const int n_ids = sc[3];

    uint32_t tmem = 0;
    if (warp != SW && warp != SW + 2) {
        if (warp == SW + 1) ptx::tmem_alloc(ptx::smem_u32(sc), T::TMEM_COLS);
#pragma unroll
        for (int t = 0; t < QV; ++t) {
            const int idx = tq + t * NQT;
            const int r = idx / (DH / 8), ch = idx % (DH / 8);
            if (idx < BM * (DH / 8))
                ptx::sts128(sQ + (ch >> 3) * (BM * 128) + r * 128 + (((ch & 7) ^ (r & 7)) << 4), qv[t]);
        }
        ptx::fence_proxy_async();              // generic-proxy writes of Q before the tensor core reads them
        ptx::tc_fence_before();
        ptx::named_bar_sync(2, NQT);
        ptx::tc_fence_after();
        tmem = *reinterpret_cast<volatile uint32_t *>(sc);
    }

    // what a softmax thread carries out of the key loop for its row
    float fin_m = -CUDART_INF_F, fin_l = 0.f;
    bool fin_have = false, fin_any = false;

    if (warp == SW || warp == SW + 2) {
        // ======================= the two loader warps: one for K tiles, one for V tiles =======================
        // (separate rings: a K slot is free again as soon as its Q K^T is done, long before the V slot of
        // the same tile, so the next K tile can be on its way a whole tile earlier)
        const bool is_k = warp == SW;
        const uint32_t full0 = is_k ? k_full : v_full, empty0 = is_k ? k_empty : v_empty, dst0 = is_k ? sK : sV;
        const CUtensorMap *tm = is_k ? &tm_ks : &tm_vs;
        const CUtensorMap *tm_own = is_k ? &tm_ko : &tm_vo;
        int it = 0;
        bool ok = true;
        for (int n = 0; n < n_ids && ok; ++n) {
            const int cur = ids[n], r0 = rng0[n], r1 = rng1[n];
            if (cur < 0) {
                // a tile of own keys: one box of OWN rows per unit (a unit past the batch reads as zeros)
                const int s = it % KV_STAGES;
                if (!__all_sync(0xffffffffu, ptx::mbar_wait(empty0 + 8 * s, ((it / KV_STAGES) & 1) ^ 1))) {
                    if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
                    ok = false;
                    break;
                }
                if (ptx::elect_one()) {
                    ptx::mbar_arrive_expect_tx(full0 + 8 * s, T::KV_BYTES);
                    for (int i = 0; i < BN / OWN; ++i) {
                        const int u = unit0 + (-1 - cur) * (BN / OWN) + i;
                        const int y = u < p.n_units ? (u * p.Hkv + h) * p.cap : p.n_units * p.Hkv * p.cap;
#pragma unroll
                        for (int hh = 0; hh < T::HALVES; ++hh)
                            ptx::tma_load_2d(dst0 + s * T::KV_BYTES + hh * (BN * 128) + i * (OWN * 128), tm_own, hh * 64, y, full0 + 8 * s);
                    }
                }
                __syncwarp();
                ++it;
                continue;
            }
            const int row_base = (cur * p.Hkv + h) * p.cap_sh;
            for (int k0 = r0; k0 < r1; k0 += BN, ++it) {
                const int s = it % KV_STAGES;
                if (!__all_sync(0xffffffffu, ptx::mbar_wait(empty0 + 8 * s, ((it / KV_STAGES) & 1) ^ 1))) {
                    if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
                    ok = false;
                    break;                     // stop loading; the other warps run out on their own bounded waits
                }
                if (ptx::elect_one()) {
                    ptx::mbar_arrive_expect_tx(full0 + 8 * s, T::KV_BYTES);
#pragma unroll
                    for (int hh = 0; hh < T::HALVES; ++hh)
                        ptx::tma_load_2d(dst0 + s * T::KV_BYTES + hh * (BN * 128), tm, hh * 64, row_base + k0, full0 + 8 * s);
                }
                __syncwarp();
            }
        }
    } else if (warp == SW + 1) {
        // ======================= MMA warp =======================
        constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(BM, BN, false, false);
        constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16(BM, DH, false, true);
        int n_tiles = 0;
        for (int n = 0; n < n_ids; ++n) n_tiles += (rng1[n] - rng0[n] + BN - 1) / BN;
        bool ok = true;
        auto issue_qk = [&](int i) {           // S[i % 2] = Q K_i^T
            const int s = i % KV_STAGES, b = i & 1;
            bool good = ptx::mbar_wait(k_full + 8 * s, (i / KV_STAGES) & 1);
            if (good && i >= 2) good = ptx::mbar_wait(s_free + 8 * b, ((i - 2) >> 1) & 1);
            if (!__all_sync(0xffffffffu, good)) return false;
            ptx::tc_fence_after();
            if (ptx::elect_one()) {
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    const uint64_t a = ptx::umma_desc_sw128(sQ + (ks >> 2) * (BM * 128) + (ks & 3) * 32, 0, 1024);
                    const uint64_t bdesc = ptx::umma_desc_sw128(sK + s * T::KV_BYTES + (ks >> 2) * (BN * 128) + (ks & 3) * 32, 0, 1024);
                    ptx::umma_bf16(tmem + b * BN, a, bdesc, idesc_qk, ks != 0);
                }
                ptx::umma_commit(s_ready + 8 * b);
                ptx::umma_commit(k_empty + 8 * s);             // this K tile has been read
            }
            __syncwarp();
            return true;
        };
        if (n_tiles > 0) ok = issue_qk(0);
        for (int i = 0; i < n_tiles && ok; ++i) {
            if (i + 1 < n_tiles) ok = issue_qk(i + 1);
            if (!ok) break;
            const int s = i % KV_STAGES;
            bool good = ptx::mbar_wait(p_ready, i & 1);
            if (good) good = ptx::mbar_wait(v_full + 8 * s, (i / KV_STAGES) & 1);
            if (!__all_sync(0xffffffffu, good)) { ok = false; break; }
            ptx::tc_fence_after();
            if (ptx::elect_one()) {
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk) {     // 16 keys per MMA
                    const uint64_t a = ptx::umma_desc_sw128(sP + (kk >> 2) * (BM * 128) + (kk & 3) * 32, 0, 1024);
                    // V tile: rows = keys (the K index), 128 bytes = 64 features (the N index): N-major operand
                    const uint64_t bdesc = ptx::umma_desc_sw128(sV + s * T::KV_BYTES + kk * (16 * 128), BN * 128, 1024);
                    ptx::umma_bf16(tmem + T::COL_O, a, bdesc, idesc_pv, (i | kk) != 0);
                }
                ptx::umma_commit(v_empty + 8 * s);
                ptx::umma_commit(p_free);
            }
            __syncwarp();
        }
        if (!ok && lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
    } else {
        // ======================= softmax warps: two threads per query row =======================
        const int quad = warp & 3, hf = warp >> 2;                 // TMEM lane quadrant; which CH keys of a tile
        const int row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int my_sid = sid[row];
        constexpr int RP = DH / 32 < KP ? DH / 32 : KP;            // threads of a row that move its accumulator, 32 or more columns each
        float m_ref = -CUDART_INF_F, l_half = 0.f;                 // m_ref is kept identical in all threads of a row
        int it = 0;
        bool ok = true;
        // After a wait has run out (ok = false) the loop goes on without waiting, so that the warps
        // keep meeting at the named barrier; the results are then void and the status says so.
        for (int n = 0; n < n_ids; ++n) {
            const int cur = ids[n], r0 = rng0[n], r1 = rng1[n];
            const bool own = cur < 0;                              // a tile of own keys: OWN rows of each of BN / OWN units
            bool active = (my_sid == cur);
            int own_lo = 0, own_hi = 0;                            // my valid keys within my part of an own tile
            bool own_clear = false;                                // some unit of the tile ends before its box of rows does
            if (own) {
                for (int i = 0; i < BN / OWN; ++i) {
                    const int uu = (-1 - cur) * (BN / OWN) + i;
                    own_clear |= uu < upt && unit0 + uu < p.n_q && ulen[uu] < OWN;
                }
                const int ur = row / G, blk = ur % (BN / OWN);     // my unit in the row tile, its block of keys in its tile
                const bool mine = row < upt * G && my_sid != -2 && ur / (BN / OWN) == -1 - cur;
                active = mine && ulen[ur] > 0;
                if (active && blk / (CH / OWN) == hf) {
                    own_lo = (blk % (CH / OWN)) * OWN;
                    own_hi = own_lo + ulen[ur];
                }
            }
            for (int k0 = r0; k0 < r1; k0 += BN, ++it) {
                const int b = it & 1, st = it % KV_STAGES;
                // keys [lo, hi) of my half are in range (hi may be <= lo)
                const int lo = own ? own_lo : 0, hi = own ? own_hi : min(BN, r1 - k0) - hf * CH;
                if (ok && !__all_sync(0xffffffffu, ptx::mbar_wait(s_ready + 8 * b, (it >> 1) & 1))) ok = false;
                ptx::tc_fence_after();
                uint32_t sr[CH];
#pragma unroll
                for (int c0 = 0; c0 < CH; c0 += 32)
                    ptx::tmem_ld_32x32(tmem + lane_base + b * BN + hf * CH + c0, *reinterpret_cast<uint32_t(*)[32]>(&sr[c0]));
                ptx::tmem_ld_wait();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(s_free + 8 * b);          // the tensor pipe may overwrite this S

                // four running maxima (and, below, four running sums): one chain of 64 dependent operations
                // would cost this thread more than the arithmetic itself
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
                if (lo == 0 && hi >= CH) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const float v = __uint_as_float(sr[c]) * p.scale_log2;
                        sr[c] = __float_as_uint(v);
                        mx4[c & 3] = fmaxf(mx4[c & 3], v);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const float v = (c >= lo && c < hi) ? __uint_as_float(sr[c]) * p.scale_log2 : -CUDART_INF_F;
                        sr[c] = __float_as_uint(v);
                        mx4[c & 3] = fmaxf(mx4[c & 3], v);
                    }
                }
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                // the two threads of a row exchange their maxima; a row whose maximum outgrows its reference
                // by more than the gap makes the whole CTA rescale its accumulators
                xch_m[(b * KP + hf) * BM + row] = mx;
                if (active && m_ref != -CUDART_INF_F && mx > m_ref + RESCALE_GAP) sc[1 + b] = 1;
                ptx::named_bar_sync(1, SW * 32);
#pragma unroll
                for (int o = 1; o < KP; ++o) mx = fmaxf(mx, xch_m[(b * KP + (hf ^ o)) * BM + row]);
                const bool rescale = sc[1 + b] != 0;
                float corr = 1.f;
                if (active) {
                    if (m_ref == -CUDART_INF_F) {
                        m_ref = mx;                                        // nothing accumulated for this row yet
                    } else if (mx > m_ref + RESCALE_GAP) {
                        corr = exp2f(m_ref - mx);
                        m_ref = mx;
                    }
                }
                // the previous P V must be done before P is overwritten (and before O is touched)
                if (ok && it > 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(p_free, (it - 1) & 1))) ok = false;
                if (rescale) {
                    ptx::tc_fence_after();
#pragma unroll 1
                    for (int c0 = 0; c0 < DH / RP && hf < RP; c0 += 32) {  // my part of the row's accumulator
                        uint32_t orow[32];
                        ptx::tmem_ld_32x32(tmem + lane_base + T::COL_O + hf * (DH / RP) + c0, orow);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) orow[e] = __float_as_uint(__uint_as_float(orow[e]) * corr);
                        ptx::tmem_st_32x32(tmem + lane_base + T::COL_O + hf * (DH / RP) + c0, orow);
                    }
                    ptx::tmem_st_wait();
                    l_half *= corr;
                    ptx::named_bar_sync(1, SW * 32);                       // every reader of the flag is past it
                    if (threadIdx.x == 0) sc[1 + b] = 0;
                }
                // rows of V past the end of the range may hold anything: clear them (P is 0 there, 0 * NaN is not)
                const int tile_valid = min(BN, r1 - k0);
                if (own) {
                    if (own_clear) {                                       // every row at or past its unit's length, unit by unit
                        if (ok && !__all_sync(0xffffffffu, ptx::mbar_wait(v_full + 8 * st, (it / KV_STAGES) & 1))) ok = false;
                        for (int idx = threadIdx.x; idx < BN * T::HALVES * 8; idx += SW * 32) {
                            const int r = idx / (T::HALVES * 8), c16 = idx % (T::HALVES * 8);
                            const int uu = (-1 - cur) * (BN / OWN) + r / OWN;
                            if (r % OWN >= (uu < BM ? ulen[uu] : 0))
                                ptx::sts128(sV + st * T::KV_BYTES + (c16 >> 3) * (BN * 128) + r * 128 + ((c16 & 7) << 4),
                                            make_uint4(0u, 0u, 0u, 0u));
                        }
                    }
                } else if (tile_valid < BN) {
                    if (ok && !__all_sync(0xffffffffu, ptx::mbar_wait(v_full + 8 * st, (it / KV_STAGES) & 1))) ok = false;
                    for (int idx = threadIdx.x; idx < (BN - tile_valid) * T::HALVES * 8; idx += SW * 32) {
                        const int r = tile_valid + idx / (T::HALVES * 8), c16 = idx % (T::HALVES * 8);
                        ptx::sts128(sV + st * T::KV_BYTES + (c16 >> 3) * (BN * 128) + r * 128 + ((c16 & 7) << 4),
                                    make_uint4(0u, 0u, 0u, 0u));
                    }
                }
                // probabilities of my 64 keys, bf16, into the swizzled P tile (K-major: 64 keys per 128-byte row)
                float ls4[4] = {0.f, 0.f, 0.f, 0.f};
                // (a 128-byte row of P holds 64 keys: my CH keys start at 16-byte chunk pc0 of row `row` of half ph)
                constexpr int CPH = 64 / CH;                               // key parts per 64-key half
                const int ph = hf / CPH, pc0 = (hf % CPH) * (CH / 8);
                const uint32_t prow = sP + ph * (BM * 128) + row * 128;
                if (active) {
#pragma unroll
                    for (int ch = 0; ch < CH / 8; ++ch) {
                        float e[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            e[j] = exp2f(__uint_as_float(sr[ch * 8 + j]) - m_ref);
                            ls4[j & 3] += e[j];
                        }
                        ptx::sts128(prow + (((pc0 + ch) ^ (row & 7)) << 4),
                                    make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7])));
                    }
                } else {
#pragma unroll
                    for (int ch = 0; ch < CH / 8; ++ch) ptx::sts128(prow + (((pc0 + ch) ^ (row & 7)) << 4), make_uint4(0u, 0u, 0u, 0u));
                }
                l_half += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
                ptx::fence_proxy_async();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(p_ready);
            }
        }
        // ---- what the row carries out: reference maximum and the sum over both halves
        xch_l[hf * BM + row] = l_half;
        ptx::named_bar_sync(1, SW * 32);
        float l_sum = l_half;
#pragma unroll
        for (int o = 1; o < KP; ++o) l_sum += xch_l[(hf ^ o) * BM + row];
        if (ok && it > 0) ok = __all_sync(0xffffffffu, ptx::mbar_wait(p_free, (it - 1) & 1));
        if (!ok && lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
        ptx::tc_fence_after();
        fin_have = ok && it > 0 && l_sum > 0.f;
        fin_any = it > 0;
        fin_m = m_ref;
        fin_l = l_sum;
    }

    // ---- the key ranges of one row tile are the CTAs of one cluster.  Each CTA stages its rows
    // (acc, m, l) in its own shared memory; when every CTA of the cluster is done with its tile buffers,
    // one bulk copy per peer moves the rows that peer owns into its receive buffer (completion counted on
    // the peer's mbarrier); every CTA then merges the rows it owns by log-sum-exp from its own shared
    // memory and writes one partial per query head.
    const uint32_t stage_a = base, recv_a = base + BM * RS * 4;    // stage [BM][RS]; receive [C sources][rows_per][RS]
    if (warp < SW) {
        // every MMA and every load of this CTA is done, so its tile buffers can serve as the staging area
        const int quad = warp & 3, hf = warp >> 2;
        const int row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        float *stage = reinterpret_cast<float *>(gen) + (size_t)row * RS;
        constexpr int RP = DH / 32 < KP ? DH / 32 : KP;
#pragma unroll 1
        for (int c0 = hf * (DH / RP); c0 < (hf + 1) * (DH / RP) && hf < RP; c0 += 32) {
            uint32_t orow[32];
            if (fin_any) {                                                  // O was written by at least one P V
                ptx::tmem_ld_32x32(tmem + lane_base + T::COL_O + c0, orow);
                ptx::tmem_ld_wait();
            }
#pragma unroll
            for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4 *>(stage + c0 + e) =
                    fin_have ? make_float4(__uint_as_float(orow[e]), __uint_as_float(orow[e + 1]), __uint_as_float(orow[e + 2]),
                                           __uint_as_float(orow[e + 3]))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (hf == 0)
            *reinterpret_cast<float4 *>(stage + DH) =
                make_float4(fin_have ? fin_m : -CUDART_INF_F, fin_have ? fin_l : 0.f, 0.f, 0.f);
        ptx::fence_proxy_async();                                  // the bulk copies below read what was staged here
    }
    ptx::tc_fence_before();
    ptx::cluster_sync();                                           // staged everywhere; receive buffers are free
    if (warp == SW && ptx::elect_one()) {
        const uint32_t bytes = rows_per * RS * 4;
        for (int o = 0; o < C; ++o)
            if (o != part)
                ptx::bulk_copy_to_peer(ptx::map_cluster(recv_a + part * bytes, o), stage_a + o * bytes, bytes,
                                       ptx::map_cluster(recv_bar, o));
    }
    const bool got = ptx::mbar_wait(recv_bar, 0);                  // the rows this CTA owns are all here
    if (!got && threadIdx.x == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
    {
        const float *stage = reinterpret_cast<const float *>(gen);
        const float *recv = stage + BM * RS;
        for (int rl = warp; rl < rows_per; rl += SP_THREADS / 32) {
            const int rr = part * rows_per + rl;
            const int i = unit0 + rr / G;
            if (rr >= upt * G || i >= p.n_q) continue;
            const float *src[8];
            float f[8];
            float M = -CUDART_INF_F;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                src[r] = r == part ? stage + (size_t)rr * RS : recv + (size_t)(r * rows_per + rl) * RS;
                f[r] = -CUDART_INF_F;
                if (r < C) {
                    const float2 ml = *reinterpret_cast<const float2 *>(src[r] + DH);
                    if (ml.y > 0.f) { f[r] = ml.x; M = fmaxf(M, ml.x); }
                }
            }
            float L = 0.f;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const float l = r < C ? src[r][DH + 1] : 0.f;
                f[r] = f[r] > -CUDART_INF_F ? exp2f(f[r] - M) : 0.f;      // weight of source r (0: nothing there)
                L += l * f[r];
            }
            constexpr int NK = (DH + 127) / 128;
            float4 acc[NK];
#pragma unroll
            for (int k = 0; k < NK; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            const bool mine = 4 * lane < DH || NK > 1;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (r < C) {
#pragma unroll
                    for (int k = 0; k < NK; ++k) {
                        if (4 * lane + 128 * k < DH) {
                            const float4 v = *reinterpret_cast<const float4 *>(src[r] + 4 * lane + 128 * k);
                            acc[k].x += f[r] * v.x; acc[k].y += f[r] * v.y; acc[k].z += f[r] * v.z; acc[k].w += f[r] * v.w;
                        }
                    }
                }
            }
            (void)mine;
            const size_t qh = (size_t)i * p.Hq + (size_t)h * G + rr % G;
            if (p.own_rows) {
                // the units' own keys rode along: this is the whole result of the query head
                const bool gone = sid[rr] == -2;                  // its prefix does not exist
                if (gone && lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
                const float inv = (L > 0.f && !gone) ? 1.f / L : 0.f;
#pragma unroll
                for (int k = 0; k < NK; ++k)
                    if (4 * lane + 128 * k < DH)
                        *reinterpret_cast<uint2 *>(p.out + qh * DH + 4 * lane + 128 * k) =
                            make_uint2(pack_bf16(acc[k].x * inv, acc[k].y * inv), pack_bf16(acc[k].z * inv, acc[k].w * inv));
                if (lane == 0 && p.lse) p.lse[qh] = (L > 0.f && !gone) ? (M + log2f(L)) * 0.6931471805599453f : -CUDART_INF_F;
                continue;
            }
            float *out = p.partials + qh * (DH + 2);
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                if (4 * lane + 128 * k < DH) {
                    *reinterpret_cast<float2 *>(out + 4 * lane + 128 * k) = make_float2(acc[k].x, acc[k].y);
                    *reinterpret_cast<float2 *>(out + 4 * lane + 128 * k + 2) = make_float2(acc[k].z, acc[k].w);
                }
            }
            if (lane == 0) { out[DH] = M; out[DH + 1] = L; }
        }
    }
    // Every copy out of this CTA's staging area has landed once its peers are past their own receive wait, which
    // is where they come from: nothing but the order of arrival is needed of this barrier, no flush of the
    // results written just before it.
    ptx::cluster_sync_relaxed();
    if (warp == SW + 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, T::TMEM_COLS);
    }
}

template <int DH>
cudaError_t run(photon_ctx *ctx, AttnParams p, cudaStream_t st, long long *launches) {
    using T = SpTile<DH>;
    static size_t smem_set[kMaxDevices] = {};
    if (const cudaError_t e = ensure_dynamic_smem(shared_prefix_kernel<DH>, T::SMEM, ctx->device, smem_set)) return e;
    const int G = p.Hq / p.Hkv;
    const int upt = BM / G;
    const int groups = (p.n_q + upt - 1) / upt;
    const CUtensorMap *t;
    CUtensorMap mks, mvs, mko, mvo;
    if (!(t = ctx->tmaps.get(p.ks, (uint64_t)p.n_shared * p.Hkv * p.cap_sh, DH, BN))) return cudaErrorInvalidValue;
    mks = *t;
    if (!(t = ctx->tmaps.get(p.vs, (uint64_t)p.n_shared * p.Hkv * p.cap_sh, DH, BN))) return cudaErrorInvalidValue;
    mvs = *t;
    // the units' own caches in boxes of OWN rows (used when their keys ride along)
    if (!(t = ctx->tmaps.get(p.k, (uint64_t)p.n_units * p.Hkv * p.cap, DH, OWN))) return cudaErrorInvalidValue;
    mko = *t;
    if (!(t = ctx->tmaps.get(p.v, (uint64_t)p.n_units * p.Hkv * p.cap, DH, OWN))) return cudaErrorInvalidValue;
    mvo = *t;
    const cudaError_t e = launch_dependent(shared_prefix_kernel<DH>, dim3(groups * p.Hkv * p.splits_sh), dim3(SP_THREADS), T::SMEM, st,
                                           p.splits_sh /* the key ranges of a row tile form a cluster */, p, mks, mvs, mko, mvo);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

int shared_prefix_units_per_cta(int G) { return BM / G; }
int shared_prefix_own_rows() { return OWN; }

cudaError_t launch_shared_prefix_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                                           long long *launches) {
    return p.dh == 64 ? run<64>(ctx, p, st, launches) : run<128>(ctx, p, st, launches);
}
