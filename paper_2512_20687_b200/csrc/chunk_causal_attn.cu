// The local decoder's attention at many positions of a chunk at once (the
// teacher-forced form of Eq. 6): position t of the concatenated sequence
// [U ; X_<j] attends positions 0..t of its own chunk buffer under the standard
// causal mask described below Eq. 7.  A problem is at most 64 x 64, so the work
// is a stream of small dense tiles: HBM-bound, with the arithmetic on the
// tensor cores (mma.sync m16n8k16, bf16 in, fp32 out) because the CUDA cores
// could not keep up with the memory system at 12 flop per byte.
//
// A warp owns one (chunk, KV head).  It copies that pair's K and V rows (two
// contiguous runs) and one tile of 16 query rows at a time into its private,
// XOR-swizzled slice of shared memory with 16-byte asynchronous copies, all
// issued before the first wait; rows that do not exist are zero-filled by the
// copy itself.  Per query tile: S = Q K^T from ldmatrix fragments, mask and
// softmax in registers in the base-2 domain, the probabilities repacked as the
// A operand of P V, the result normalised, staged through the query tile's slot
// and written with 16-byte coalesced stores.  The query heads of a group reuse
// the resident K and V; the next query tile is in flight while one is computed.
// Warps never wait on each other, so there is no barrier and no spin-wait here.
#include <math_constants.h>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int CC_WARPS = 4;                 // (chunk, KV head) pairs per CTA

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
    const int bytes = valid ? 16 : 0;       // 0: the 16 bytes at dst are zero-filled, src is not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
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
    static constexpr int KROWS = KT * 16;
    static constexpr int WARP_BYTES = (2 * KROWS + 32) * ROWB;   // K, V, two query tiles
};

// byte offset of 16-byte piece `piece` of row `row`: the piece index is XORed with the row's low bits,
// so that the 8 rows of an ldmatrix tile (and the rows of a fragment store) fall on different banks
template <int ROWB>
__device__ __forceinline__ uint32_t swz(int row, int piece) {
    return (uint32_t)(row * ROWB + ((piece ^ (row & 7)) << 4));
}

template <int DH, int KT>
__global__ void __launch_bounds__(CC_WARPS * 32)
chunk_causal_attn_kernel(const CausalParams p) {
    using S = Shape<DH, KT>;
    constexpr int ROWB = S::ROWB, CPR = S::CPR, RPI = S::RPI;
    extern __shared__ __align__(128) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * CC_WARPS + warp;
    if (item >= (long long)p.n * p.Hkv) return;
    const int kvh = (int)(item % p.Hkv);
    const int i = (int)(item / p.Hkv);
    const int G = p.Hq / p.Hkv;
    const int lrow = lane / CPR, piece = lane % CPR;      // this lane's part of a warp-wide row copy

    const uint32_t sK = ptx::smem_u32(smem) + (uint32_t)warp * S::WARP_BYTES;
    const uint32_t sV = sK + S::KROWS * ROWB, sQ = sV + S::KROWS * ROWB;

    const int u = p.slot ? p.slot[i] : i;
    const bool bad = u < 0 || u >= p.n_units;
    if (bad && lane == 0) atomicOr(p.status, PHOTON_DEV_BAD_INDEX);
    const int len = bad ? 0 : max(0, min(__ldg(p.len + u), p.cap));
    const int MT = (p.R + 15) >> 4;                        // query tiles per head
    const int n_jobs = G * MT;
    const int n_keys = p.row0 < len ? min(len, p.row0 + p.R) : 0;   // rows any query of this call can see
    const int kt_all = (n_keys + 15) >> 4;

    // query row t of head g of this group / its output row
    auto row_ptr = [&](const bf16 *base, int g, int t) {
        return base + (((size_t)i * p.R + t) * p.Hq + (size_t)kvh * G + g) * DH + piece * 8;
    };
    auto store_tile = [&](int g, int mt, uint32_t src, bool from_smem) {
#pragma unroll
        for (int rr = 0; rr < 16; rr += RPI) {
            const int row = rr + lrow, t = mt * 16 + row;
            if (t >= p.R) continue;
            uint4 val = make_uint4(0u, 0u, 0u, 0u);
            if (from_smem && p.row0 + t < len) val = lds128(src + swz<ROWB>(row, piece));
            *reinterpret_cast<uint4 *>(const_cast<bf16 *>(row_ptr(p.out, g, t))) = val;
        }
    };
    if (n_keys == 0) {                                     // nothing exists yet (or a bad slot): zero rows
        for (int j = 0; j < n_jobs; ++j) store_tile(j / MT, j % MT, 0u, false);
        return;
    }

    auto load_q = [&](int j) {
        const int g = j / MT, mt = j % MT;
        const uint32_t dst = sQ + (uint32_t)(j & 1) * 16 * ROWB;
#pragma unroll
        for (int rr = 0; rr < 16; rr += RPI) {
            const int row = rr + lrow, t = mt * 16 + row;
            const bool ok = t < p.R && p.row0 + t < len;
            cp_async16(dst + swz<ROWB>(row, piece), row_ptr(p.q, g, ok ? t : 0), ok);
        }
    };
    auto load_kv = [&](const bf16 *src, uint32_t dst) {
        const bf16 *base = src + ((size_t)u * p.Hkv + kvh) * p.cap * DH + piece * 8;
        for (int rr = 0; rr < kt_all * 16; rr += RPI) {
            const int row = rr + lrow;
            const bool ok = row < n_keys;
            cp_async16(dst + swz<ROWB>(row, piece), base + (size_t)(ok ? row : 0) * DH, ok);
        }
    };
    load_kv(p.k, sK);
    load_q(0);
    cp_async_commit();
    load_kv(p.v, sV);
    cp_async_commit();

    const int gq = lane >> 2, tq = lane & 3;
    for (int j = 0; j < n_jobs; ++j) {
        __syncwarp();                                      // the other query slot is no longer read
        if (j + 1 < n_jobs) load_q(j + 1);
        cp_async_commit();                                 // (possibly empty: keeps the group count uniform)
        const int g = j / MT, mt = j % MT;
        const int q_lo = p.row0 + mt * 16;                 // position of the tile's first row
        const uint32_t qb = sQ + (uint32_t)(j & 1) * 16 * ROWB;
        if (q_lo >= len) {                                 // none of these positions exists yet
            store_tile(g, mt, 0u, false);
            continue;
        }
        // groups so far: {K, Q0}, {V}, {Q1}, ..., {Q(j+1)}; all but the newest must have landed, and for the
        // first job K and Q0 are enough to start with
        if (j == 0) cp_async_wait<2>(); else cp_async_wait<1>();
        __syncwarp();
        const int kt_hi = min(kt_all, ((q_lo + 15) >> 4) + 1);   // 16-key tiles this query tile can see

        // ---- S = Q K^T ----
        float s[2 * KT][4];
#pragma unroll
        for (int nt = 0; nt < 2 * KT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            uint32_t a[4];
            {
                const int row = (lane & 7) + ((lane >> 3) & 1) * 8;
                ptx::ldmatrix_x4(a, qb + swz<ROWB>(row, ks * 2 + (lane >> 4)));
            }
#pragma unroll
            for (int kp = 0; kp < KT; ++kp) {
                if (kp >= kt_hi) continue;
                uint32_t b[4];
                const int row = kp * 16 + (lane & 7) + (lane >> 4) * 8;
                ptx::ldmatrix_x4(b, sK + swz<ROWB>(row, ks * 2 + ((lane >> 3) & 1)));
                ptx::mma_bf16_16816(s[2 * kp], a, b[0], b[1]);
                ptx::mma_bf16_16816(s[2 * kp + 1], a, b[2], b[3]);
            }
        }
        // ---- causal mask and softmax (rows gq and gq + 8 of the tile) ----
        float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
        for (int nt = 0; nt < 2 * KT; ++nt) {
            if (nt >= 2 * kt_hi) continue;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = nt * 8 + 2 * tq + (e & 1), row = gq + (e >> 1) * 8;
                const float x = key <= q_lo + row ? s[nt][e] * p.scale_log2 : -CUDART_INF_F;
                s[nt][e] = x;
                mx[e >> 1] = fmaxf(mx[e >> 1], x);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));   // finite: key 0 is always visible
        }
        float sum[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < 2 * KT; ++nt) {
            if (nt >= 2 * kt_hi) continue;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float w = exp2f(s[nt][e] - mx[e >> 1]);
                s[nt][e] = w;
                sum[e >> 1] += w;
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 1);
            sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 2);
        }
        // ---- O = P V ----
        if (j == 0) { cp_async_wait<1>(); __syncwarp(); }   // V has landed
        float o[DH / 8][4];
#pragma unroll
        for (int nt = 0; nt < DH / 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
#pragma unroll
        for (int kp = 0; kp < KT; ++kp) {
            if (kp >= kt_hi) continue;
            uint32_t a[4];
            a[0] = pack_bf16(s[2 * kp][0], s[2 * kp][1]);
            a[1] = pack_bf16(s[2 * kp][2], s[2 * kp][3]);
            a[2] = pack_bf16(s[2 * kp + 1][0], s[2 * kp + 1][1]);
            a[3] = pack_bf16(s[2 * kp + 1][2], s[2 * kp + 1][3]);
#pragma unroll
            for (int np = 0; np < DH / 16; ++np) {
                uint32_t b[4];
                const int row = kp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ptx::ldmatrix_x4_trans(b, sV + swz<ROWB>(row, np * 2 + (lane >> 4)));
                ptx::mma_bf16_16816(o[2 * np], a, b[0], b[1]);
                ptx::mma_bf16_16816(o[2 * np + 1], a, b[2], b[3]);
            }
        }
        // ---- normalise, stage through the query tile's slot, store rows ----
        const float inv0 = 1.f / sum[0], inv1 = 1.f / sum[1];
        __syncwarp();                                      // every lane is done reading the query tile
#pragma unroll
        for (int nt = 0; nt < DH / 8; ++nt) {
            sts32(qb + swz<ROWB>(gq, nt) + tq * 4, pack_bf16(o[nt][0] * inv0, o[nt][1] * inv0));
            sts32(qb + swz<ROWB>(gq + 8, nt) + tq * 4, pack_bf16(o[nt][2] * inv1, o[nt][3] * inv1));
        }
        __syncwarp();
        store_tile(g, mt, qb, true);
    }
    cp_async_wait<0>();
}

template <int DH, int KT>
cudaError_t launch(photon_ctx *ctx, const CausalParams &p, cudaStream_t st, long long *launches) {
    static size_t attr_set[kMaxDevices] = {};
    constexpr size_t smem = (size_t)CC_WARPS * Shape<DH, KT>::WARP_BYTES;
    cudaError_t e = ensure_dynamic_smem(chunk_causal_attn_kernel<DH, KT>, smem, ctx->device, attr_set);
    if (e != cudaSuccess) return e;
    const long long items = (long long)p.n * p.Hkv;
    // a plain launch, like the single-query chunk kernel: many waves of short CTAs
    chunk_causal_attn_kernel<DH, KT><<<(unsigned)((items + CC_WARPS - 1) / CC_WARPS), CC_WARPS * 32, smem, st>>>(p);
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
