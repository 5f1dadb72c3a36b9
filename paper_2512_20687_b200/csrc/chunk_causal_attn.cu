// The local decoder's attention at many positions of a chunk at once (the
// teacher-forced form of Eq. 6): position t of the concatenated sequence
// [U ; X_<j] attends positions 0..t of its own chunk buffer under the standard
// causal mask described below Eq. 7.  A problem is at most 64 x 64, so the work
// is a stream of small dense tiles: HBM-bound, with the arithmetic on the
// tensor cores (mma.sync m16n8k16, bf16 in, fp32 out) because the CUDA cores
// could not keep up with the memory system at 12 flop per byte.
//
// A warp owns one (chunk, KV head) at a time and never waits on another warp:
// there is no barrier between warps and no spin-wait in this kernel.  It copies
// that pair's K and V rows (two contiguous runs) and one tile of 16 query rows
// at a time into its private, XOR-swizzled slice of shared memory with 16-byte
// asynchronous copies that run ahead of the arithmetic: the next pair's K is
// requested as soon as the last S of this pair is done, its V after the last
// P V, and each query slot is refilled two tiles ahead.  Per query tile:
// S = Q K^T from ldmatrix fragments, mask and softmax in registers in the base-2
// domain, the normalised probabilities repacked as the A operand of P V, the
// result staged through the query tile's slot with stmatrix and written with
// 16-byte coalesced stores.  The query heads of a group reuse the resident K
// and V.  On a large call pairs are handed out from a counter in global memory,
// so an SM that gets less memory bandwidth than its neighbours takes fewer.
//
// The kernel is bound by instruction issue as much as by memory, so every
// shared-memory offset that depends only on the lane is computed once, the
// copy loops are unrolled with immediate offsets, and the arithmetic is
// instantiated per number of visible key tiles instead of predicated.
#include <math_constants.h>

#include <algorithm>
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace {

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void *src, bool valid) {
    const int bytes = valid ? 16 : 0;       // 0: the 16 bytes at dst are zero-filled, src is not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void stmatrix_x4(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r0), "r"(r1),
                 "r"(r2), "r"(r3)
                 : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

// DH: head size; KT: 16-row tiles of the chunk buffer that can hold keys (cap <= 16 * KT)
template <int DH, int KT>
struct Shape {
    static constexpr int ROWB = DH * 2;                 // bytes per row
    static constexpr int CPR = DH / 8;                  // 16-byte pieces per row
    static constexpr int RPI = 32 / CPR;                // rows one warp-wide copy covers
    static constexpr int NC = 8 / RPI;                  // distinct swizzle phases of a lane's copies
    static constexpr int KROWS = KT * 16;
    static constexpr int WARP_BYTES = (2 * KROWS + 32) * ROWB;   // K, V, two query tiles
    // Warps per CTA (one CTA per SM): what shared memory holds, and no more than the register file allows.
    // A scheduler owns a quarter of the registers, so up to 8 warps may use 255 registers each and 9 to 12
    // only 168, which the short-head variants with few key tiles fit into.
    static constexpr int FIT = (227 * 1024) / WARP_BYTES;
    static constexpr int CAP = (DH == 64 && KT <= 2) ? 12 : 8;
    static constexpr int WARPS = FIT < CAP ? FIT : CAP;
};

// One unit of work of a warp: a (chunk, KV head) pair, or one query head of it when the launch splits
// the groups.  kt_all = 0 marks a pair none of whose positions exists (or a bad slot): zero rows.
struct Item {
    int i, kvh, g0;
    int u, len, n_keys, kt_all;
};

// Shared-memory layout of a slice: row r at r * ROWB, its 16-byte piece c at ((c ^ (r & 7)) << 4), so that
// the 8 rows of an ldmatrix / stmatrix tile and the rows of a warp-wide copy fall on different banks.
template <int DH, int KT>
__global__ void __launch_bounds__(Shape<DH, KT>::WARPS * 32, 1)
chunk_causal_attn_kernel(const CausalParams p) {
    using S = Shape<DH, KT>;
    constexpr int ROWB = S::ROWB, CPR = S::CPR, RPI = S::RPI, NC = S::NC;
    extern __shared__ __align__(128) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_warps = blockDim.x >> 5;
    const int G = p.Hq / p.Hkv, GJ = G / p.gsplit;        // query heads per item
    const int MT = (p.R + 15) >> 4;                        // query tiles per head
    const int J = GJ * MT;                                 // jobs (query tiles) per item
    const int total = p.n * p.Hkv * p.gsplit;             // items of this call (the host keeps it below 2^31)

    // The first item of a warp is its own index.  On a large call the rest are handed out from a counter
    // in global memory in batches of consecutive items whose size shrinks as the work runs out (half of an
    // even share of what is left, at most 16): atomics on one address complete only every few
    // nanoseconds, so there must be far fewer of them than items, while the last batches must be small
    // for the SMs to finish together.  The next batch is claimed when one is opened and read (from lane 0)
    // when that one is used up, so the counter's latency stays off the critical path.  A call with fewer
    // than 16 items per warp is dealt out round-robin instead: there the claims' latency would cost more
    // than uneven SMs do.
    const int all_warps = (int)gridDim.x * n_warps;
    const bool ticketed = total >= 16 * all_warps;
    __shared__ int warps_left;
    if (threadIdx.x == 0) warps_left = n_warps;
    __syncthreads();
    auto retire = [&]() {                                  // the last warp of the last CTA rewinds the counters
        if (!ticketed || lane != 0) return;
        if (atomicSub(&warps_left, 1) != 1) return;
        if (atomicAdd(p.work + 1, 1) == (int)gridDim.x - 1) { p.work[0] = 0; p.work[1] = 0; }
    };
    int batch = total, batch_n = 0, off = 0;               // open batch, its size, items used of it
    int pending = total, pending_n = 0;                    // next batch (valid in lane 0)
    auto claim = [&]() {
        if (lane != 0) return;
        const int left = total - all_warps - *reinterpret_cast<volatile int *>(p.work);   // may be stale: only sizes the claim
        pending_n = max(1, min(16, left / (2 * all_warps)));
        pending = all_warps + atomicAdd(p.work, pending_n);
    };
    int id0 = (int)blockIdx.x * n_warps + warp;
    if (id0 >= total) { retire(); return; }
    if (ticketed) claim();
    int strided = id0;
    auto next_id = [&]() {
        if (!ticketed) return strided = min(total, strided + all_warps);
        if (off == batch_n) {
            batch = __shfl_sync(0xffffffffu, pending, 0);
            batch_n = __shfl_sync(0xffffffffu, pending_n, 0);
            claim();
            off = 0;
        }
        return batch + off++;
    };
    int id1 = next_id(), id2 = next_id(), id3 = next_id();

    // ---- per-lane constants ----
    const int lrow = lane / CPR, piece = lane % CPR;       // this lane's part of a warp-wide row copy
    const uint32_t sK = ptx::smem_u32(smem) + (uint32_t)warp * S::WARP_BYTES;
    const uint32_t sV = sK + S::KROWS * ROWB, sQ = sV + S::KROWS * ROWB;
    // copies: row rr + lrow (rr a multiple of RPI) sits at rr * ROWB + cpo[(rr / RPI) % NC]
    uint32_t cpo[NC];
#pragma unroll
    for (int m = 0; m < NC; ++m) cpo[m] = (uint32_t)(lrow * ROWB + (((piece ^ lrow) ^ (m * RPI)) << 4));
    // fragment tiles: ldmatrix of Q (A operand) and of V (B operand, transposed) and stmatrix of O address
    // row (lane & 7) + 8 * ((lane >> 3) & 1), pieces 2 * x + (lane >> 4); ldmatrix of K (B operand) addresses
    // row (lane & 7) + 8 * (lane >> 4), pieces 2 * x + ((lane >> 3) & 1).  Piece 2x + h of row r sits at
    // ((x >> 2) << 7) + ((((x & 3) * 2 + h) ^ (r & 7)) << 4): four XOR phases per lane, the rest immediate.
    uint32_t ao[4], bo[4];
    {
        const int r7 = lane & 7, h1 = (lane >> 3) & 1, h2 = lane >> 4;
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            ao[m] = (uint32_t)((r7 + 8 * h1) * ROWB + (((m * 2 + h2) ^ r7) << 4));
            bo[m] = (uint32_t)((r7 + 8 * h2) * ROWB + (((m * 2 + h1) ^ r7) << 4));
        }
    }
    const int gq = lane >> 2, tq = lane & 3;
    const size_t q_row_stride = (size_t)p.Hq * DH;        // elements between consecutive rows of q / out

    auto where = [&](int x, int &i, int &kvh, int &g0) {
        const int per = p.Hkv * p.gsplit, rem = x % per;
        i = x / per; kvh = rem / p.gsplit; g0 = (rem % p.gsplit) * GJ;
    };
    auto get_item = [&](int x) {
        Item it;
        where(x, it.i, it.kvh, it.g0);
        it.u = p.slot ? __ldcg(p.slot + it.i) : it.i;           // index arrays through the L2: another kernel may have just written them
        const bool bad = it.u < 0 || it.u >= p.n_units;
        if (bad && lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
        it.len = bad ? 0 : max(0, min(__ldcg(p.len + it.u), p.cap));
        it.n_keys = p.row0 < it.len ? min(it.len, p.row0 + p.R) : 0;   // rows any query of this call can see
        it.kt_all = (it.n_keys + 15) >> 4;
        return it;
    };
    // this lane's piece of row (16 * mt + lrow) of query head g of chunk i, in q or out
    auto tile_ptr = [&](const bf16 *base, int i, int kvh, int g, int mt) {
        return base + (((size_t)i * p.R + mt * 16 + lrow) * p.Hq + (size_t)kvh * G + g) * DH + piece * 8;
    };
    // the query rows of job j of item x -> query slot `slot`.  Rows are fetched whether or not their
    // position exists yet (q holds all R rows of a chunk); what does not exist is zeroed at the output,
    // and rows beyond R are left as they are: a row of S, P and O depends on its own query row only.
    auto load_q = [&](int x, int j, int slot) {
        if (x >= total) return;
        int i, kvh, g0;
        where(x, i, kvh, g0);
        const int mt = j % MT;
        const bf16 *src = tile_ptr(p.q, i, kvh, g0 + j / MT, mt);
        const uint32_t dst = sQ + (uint32_t)slot * 16 * ROWB;
        const int rows = p.R - mt * 16 - lrow;             // row rr of this lane exists iff rr < rows
#pragma unroll
        for (int rr = 0; rr < 16; rr += RPI)
            if (rr < rows) cp_async16(dst + cpo[(rr / RPI) % NC] + rr * ROWB, src + rr * q_row_stride);
    };
    // K: rows >= n_keys are not fetched (their logits are replaced, not multiplied).  V: rows from n_keys
    // to the end of the last key tile are zero-filled, because a zero probability times a NaN is a NaN.
    auto load_k = [&](const Item &it) {
        const bf16 *src = p.k + ((size_t)it.u * p.Hkv + it.kvh) * p.cap * DH + lrow * DH + piece * 8;
        const int rows = it.n_keys - lrow;
#pragma unroll
        for (int rr = 0; rr < S::KROWS; rr += RPI)
            if (rr < rows) cp_async16(sK + cpo[(rr / RPI) % NC] + rr * ROWB, src + rr * DH);
    };
    auto load_v = [&](const Item &it) {
        const bf16 *src0 = p.v + ((size_t)it.u * p.Hkv + it.kvh) * p.cap * DH + piece * 8;   // row 0: always there
        const bf16 *src = src0 + lrow * DH;
        const int rows = it.n_keys - lrow, fill = it.kt_all * 16;
#pragma unroll
        for (int rr = 0; rr < S::KROWS; rr += RPI)
            if (rr < fill)
                cp_async16_zfill(sV + cpo[(rr / RPI) % NC] + rr * ROWB, rr < rows ? src + rr * DH : src0, rr < rows);
    };

    // The copies run ahead of the arithmetic in a fixed rhythm of three commit groups per job:
    //   after S of a job      {K of the next item, if this was the item's last job}
    //   after P V of a job    {V of the next item, likewise}
    //   after the job's store {the query tile two jobs ahead, into the slot just vacated}
    // so "all but the newest two groups" is always what the next consumer needs.
    Item cur = get_item(id0);
    int q_pos = 0, q_j = 0;                                // cursor of the query-tile copies: (item in hand, job)
    auto q_id = [&]() { return q_pos == 0 ? id0 : q_pos == 1 ? id1 : id2; };   // never past the third item in hand
    auto advance_q = [&]() { if (++q_j == J) { q_j = 0; ++q_pos; } };
    load_q(q_id(), q_j, 0); advance_q(); cp_async_commit();
    load_k(cur); cp_async_commit();
    load_v(cur); cp_async_commit();
    load_q(q_id(), q_j, 1); advance_q(); cp_async_commit();

    int jc = 0;                                            // jobs done by this warp: picks the query slot
    while (id0 < total) {
        Item nxt;
        if (id1 < total) nxt = get_item(id1); else { nxt = cur; nxt.kt_all = 0; nxt.n_keys = 0; }
        const int id4 = next_id();
        for (int j = 0; j < J; ++j, ++jc) {
            const int g = cur.g0 + j / MT, mt = j % MT;
            const int q_lo = p.row0 + mt * 16;             // position of the tile's first row
            const bool last = j == J - 1;
            const uint32_t qb = sQ + (uint32_t)(jc & 1) * 16 * ROWB;
            // 16-key tiles this query tile can see; 0: none of its positions exists yet
            const int kt_hi = q_lo < cur.len ? min(cur.kt_all, ((q_lo + 15) >> 4) + 1) : 0;

            // The arithmetic is instantiated per number of visible key tiles (no predicates inside); the
            // copies between its two halves exist once.
            float s[2 * KT][4];
            auto scores = [&](auto kh_tag) {
                constexpr int KH = decltype(kh_tag)::value;
                // ---- S = Q K^T ----
#pragma unroll
                for (int nt = 0; nt < 2 * KH; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    uint32_t a[4];
                    ptx::ldmatrix_x4(a, qb + ao[ks & 3] + ((ks >> 2) << 7));
#pragma unroll
                    for (int kp = 0; kp < KH; ++kp) {
                        uint32_t b[4];
                        ptx::ldmatrix_x4(b, sK + bo[ks & 3] + ((ks >> 2) << 7) + kp * 16 * ROWB);
                        ptx::mma_bf16_16816(s[2 * kp], a, b[0], b[1]);
                        ptx::mma_bf16_16816(s[2 * kp + 1], a, b[2], b[3]);
                    }
                }
                // ---- causal mask and softmax (rows gq and gq + 8 of the tile) ----
                // element e of key tile nt is key 8 nt + 2 tq + (e & 1) of row gq + 8 (e >> 1):
                // visible iff 8 nt <= lim[e]
                int lim[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) lim[e] = q_lo + gq + (e >> 1) * 8 - 2 * tq - (e & 1);
                float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                for (int nt = 0; nt < 2 * KH; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float x = nt * 8 <= lim[e] ? s[nt][e] * p.scale_log2 : -CUDART_INF_F;
                        s[nt][e] = x;
                        mx[e >> 1] = fmaxf(mx[e >> 1], x);
                    }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));   // finite: key 0 is always visible
                }
                float sum[2] = {0.f, 0.f};
#pragma unroll
                for (int nt = 0; nt < 2 * KH; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float w = exp2f(s[nt][e] - mx[e >> 1]);
                        s[nt][e] = w;
                        sum[e >> 1] += w;
                    }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 1);
                    sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 2);
                }
                // the probabilities are normalised before P V: fewer multiplications than scaling O
                const float inv0 = 1.f / sum[0], inv1 = 1.f / sum[1];
#pragma unroll
                for (int nt = 0; nt < 2 * KH; ++nt) {
                    s[nt][0] *= inv0; s[nt][1] *= inv0; s[nt][2] *= inv1; s[nt][3] *= inv1;
                }
            };
            auto output = [&](auto kh_tag) {
                constexpr int KH = decltype(kh_tag)::value;
                // ---- O = P V, staged through the query tile's slot ----
                float o[DH / 8][4];
#pragma unroll
                for (int nt = 0; nt < DH / 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
#pragma unroll
                for (int kp = 0; kp < KH; ++kp) {
                    uint32_t a[4];
                    a[0] = pack_bf16(s[2 * kp][0], s[2 * kp][1]);
                    a[1] = pack_bf16(s[2 * kp][2], s[2 * kp][3]);
                    a[2] = pack_bf16(s[2 * kp + 1][0], s[2 * kp + 1][1]);
                    a[3] = pack_bf16(s[2 * kp + 1][2], s[2 * kp + 1][3]);
#pragma unroll
                    for (int np = 0; np < DH / 16; ++np) {
                        uint32_t b[4];
                        ptx::ldmatrix_x4_trans(b, sV + ao[np & 3] + ((np >> 2) << 7) + kp * 16 * ROWB);
                        ptx::mma_bf16_16816(o[2 * np], a, b[0], b[1]);
                        ptx::mma_bf16_16816(o[2 * np + 1], a, b[2], b[3]);
                    }
                }
                __syncwarp();                              // every lane has read the query tile (and its V fragments)
#pragma unroll
                for (int np = 0; np < DH / 16; ++np)
                    stmatrix_x4(qb + ao[np & 3] + ((np >> 2) << 7), pack_bf16(o[2 * np][0], o[2 * np][1]),
                                pack_bf16(o[2 * np][2], o[2 * np][3]), pack_bf16(o[2 * np + 1][0], o[2 * np + 1][1]),
                                pack_bf16(o[2 * np + 1][2], o[2 * np + 1][3]));
            };
            auto dispatch = [&](auto &&f) {
                switch (kt_hi) {
                    case 0: break;
                    case 1: f(std::integral_constant<int, 1>{}); break;
                    case 2: if constexpr (KT >= 2) f(std::integral_constant<int, 2>{}); break;
                    case 3: if constexpr (KT >= 3) f(std::integral_constant<int, 3>{}); break;
                    default: if constexpr (KT >= 4) f(std::integral_constant<int, 4>{}); break;
                }
            };

            cp_async_wait<2>();                            // K of this item and this job's query tile are here
            __syncwarp();
            dispatch(scores);
            __syncwarp();                                  // every lane has read its K fragments
            if (last) load_k(nxt);
            cp_async_commit();

            cp_async_wait<2>();                            // V of this item is here
            __syncwarp();
            dispatch(output);
            __syncwarp();                                  // V has been read; the staged tile is complete
            if (last) load_v(nxt);
            cp_async_commit();

            // ---- store rows: 16-byte pieces, a position that does not exist yet gives a zero row ----
            bf16 *dst = const_cast<bf16 *>(tile_ptr(p.out, cur.i, cur.kvh, g, mt));
            const int rows = p.R - mt * 16 - lrow;         // rows of the call
            const int have = kt_hi > 0 ? cur.len - q_lo - lrow : 0;    // rows whose position exists
#pragma unroll
            for (int rr = 0; rr < 16; rr += RPI) {
                if (rr >= rows) continue;
                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                if (rr < have) val = lds128(qb + cpo[(rr / RPI) % NC] + rr * ROWB);
                *reinterpret_cast<uint4 *>(dst + rr * q_row_stride) = val;
            }
            __syncwarp();                                  // the slot has been read out
            load_q(q_id(), q_j, jc & 1); advance_q();
            cp_async_commit();
        }
        cur = nxt;
        id0 = id1; id1 = id2; id2 = id3; id3 = id4;
        --q_pos;
    }
    cp_async_wait<0>();
    retire();
}

template <int DH, int KT>
cudaError_t launch(photon_ctx *ctx, CausalParams p, cudaStream_t st, long long *launches) {
    static size_t attr_set[kMaxDevices] = {};
    using S = Shape<DH, KT>;
    constexpr int W = S::WARPS;
    const int G = p.Hq / p.Hkv;
    // few chunks: give each query head of a group to a warp of its own (K and V then come from L2 for the others)
    p.gsplit = ((long long)p.n * p.Hkv < 2ll * ctx->sm_count * W) ? G : 1;
    const long long items = (long long)p.n * p.Hkv * p.gsplit;
    if (items >= (1ll << 31) - 65536) return cudaErrorInvalidValue;      // item indices are 32-bit
    p.work = ctx->work;
    // one persistent CTA per SM; a small call is spread over the SMs with fewer warps per CTA
    int w = W;
    if (items < (long long)ctx->sm_count * W) w = (int)std::max(1ll, (items + ctx->sm_count - 1) / ctx->sm_count);
    const unsigned grid = (unsigned)std::min<long long>(ctx->sm_count, (items + w - 1) / w);
    cudaError_t e = ensure_dynamic_smem(chunk_causal_attn_kernel<DH, KT>, (size_t)W * S::WARP_BYTES, ctx->device, attr_set);
    if (e != cudaSuccess) return e;
    chunk_causal_attn_kernel<DH, KT><<<grid, w * 32, (size_t)w * S::WARP_BYTES, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

template <int DH>
cudaError_t pick_tiles(photon_ctx *ctx, const CausalParams &p, cudaStream_t st, long long *launches) {
    if (p.cap <= 16) return launch<DH, 1>(ctx, p, st, launches);
    if (p.cap <= 32) return launch<DH, 2>(ctx, p, st, launches);
    if (p.cap <= 48) return launch<DH, 3>(ctx, p, st, launches);
    return launch<DH, 4>(ctx, p, st, launches);
}

}  // namespace

cudaError_t launch_chunk_causal_attention(photon_ctx *ctx, const CausalParams &p, cudaStream_t st,
                                          long long *launches) {
    if (p.n == 0) return cudaSuccess;
    return p.dh == 64 ? pick_tiles<64>(ctx, p, st, launches) : pick_tiles<128>(ctx, p, st, launches);
}
