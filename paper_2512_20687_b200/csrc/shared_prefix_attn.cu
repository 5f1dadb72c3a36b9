// Shared-prefix phase of the coarse decode attention (Section 1: long-context,
// multi-query serving): many units (query branches) attend the same stored
// prefix, which is therefore read once for a whole group of units.
//
// CTA = (group of units, KV head, key range of the prefix).  The K/V tiles of
// the range stream through a TMA-fed, 128-byte-swizzled shared-memory ring; each
// of the four consumer warps owns 16 query rows (16/G units x G heads) and runs
// them against every key of a tile on tensor cores with an fp32 online softmax
// in the base-2 domain, so the prefix leaves HBM once and L2 feeds the other
// groups.  Every (query head, key range) leaves an unnormalised partial
// (acc, m, l) at partials[(query head) * splits_sh + range]; the kernel that
// streams the units' own keys folds these partials into its result.
#include <math_constants.h>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int NW = 4;                      // consumer warps per CTA
constexpr int BN = 64;                     // keys per tile
constexpr int THREADS = (NW + 1) * 32;     // + one producer warp
constexpr int HALF_BYTES = BN * 128;       // one 64-row x 64-element swizzled box

template <int DH>
struct Tile {
    static constexpr int HALVES = DH / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;     // K (or V) tile
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int STAGES = DH == 128 ? 3 : 4;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers, flags*/ +
                                64 * 4 /*shared ids*/;
};

__device__ __forceinline__ void part_range(int L, int n_splits, int p, int &r0, int &r1) {
    // ranges start on tile boundaries so that TMA rows stay aligned to the key tiles
    const int per = ((L + n_splits - 1) / n_splits + BN - 1) / BN * BN;
    r0 = min(L, p * per);
    r1 = min(L, r0 + per);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

// One 16-key block of a tile against the warp's 16 query rows.
//   kt, vt   shared-memory addresses of the K and V tiles (swizzled boxes)
//   kb       index of the 16-key block inside the tile
//   valid    number of valid keys in the block (1..16)
//   act0/1   whether this thread's rows g and g+8 take part
template <int DH>
__device__ __forceinline__ void process_block(uint32_t kt, uint32_t vt, int kb, int valid,
                                              const uint32_t (&qa)[DH / 16][4], float (&o)[DH / 8][4],
                                              float (&m)[2], float (&l)[2], float scale_log2, int lane,
                                              bool act0, bool act1, bool hi_rows) {
    const int c = lane & 3;
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[j][e] = 0.f;

    // S = Q K^T : B fragments straight from the swizzled K tile
    {
        const int mi = lane >> 3, r8 = lane & 7;
#pragma unroll
        for (int ks2 = 0; ks2 < DH / 32; ++ks2) {
            const int cfull = ks2 * 4 + mi;                      // 16-byte chunk along dh
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int row = kb * 16 + j * 8 + r8;
                const uint32_t addr = kt + (cfull >> 3) * HALF_BYTES + row * 128 +
                                      ((((cfull & 7) ^ (row & 7))) << 4);
                uint32_t b[4];
                ptx::ldmatrix_x4(b, addr);
                ptx::mma_bf16_16816(s[j], qa[ks2 * 2], b[0], b[1]);
                ptx::mma_bf16_16816(s[j], qa[ks2 * 2 + 1], b[2], b[3]);
            }
        }
    }
    // scale, mask the tail keys
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int key = j * 8 + 2 * c + (e & 1);
            s[j][e] = key < valid ? s[j][e] * scale_log2 : -CUDART_INF_F;
        }
    // online softmax, rows g (slot 0) and g+8 (slot 1)
    float corr[2] = {1.f, 1.f};
    uint32_t pa[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int rs = 0; rs < 2; ++rs) {
        if (rs == 1 && !hi_rows) break;
        const bool act = rs ? act1 : act0;
        float mx = fmaxf(fmaxf(s[0][2 * rs], s[0][2 * rs + 1]), fmaxf(s[1][2 * rs], s[1][2 * rs + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mn = fmaxf(m[rs], mx);
        const float cr = exp2f(m[rs] - mn);
        float p0 = exp2f(s[0][2 * rs] - mn), p1 = exp2f(s[0][2 * rs + 1] - mn);
        float p2 = exp2f(s[1][2 * rs] - mn), p3 = exp2f(s[1][2 * rs + 1] - mn);
        if (act) {
            corr[rs] = cr;
            m[rs] = mn;
            l[rs] = l[rs] * cr + ((p0 + p1) + (p2 + p3));
            pa[rs] = pack_bf16(p0, p1);           // keys 2c, 2c+1
            pa[rs + 2] = pack_bf16(p2, p3);       // keys 2c+8, 2c+9
        }
    }
    // masks that clear V entries of keys past the end (they may hold anything)
    uint32_t vm0 = 0xFFFFFFFFu, vm1 = 0xFFFFFFFFu;
    if (valid < 16) {
        vm0 = (2 * c < valid ? 0x0000FFFFu : 0u) | (2 * c + 1 < valid ? 0xFFFF0000u : 0u);
        vm1 = (2 * c + 8 < valid ? 0x0000FFFFu : 0u) | (2 * c + 9 < valid ? 0xFFFF0000u : 0u);
    }
    // O = O * corr + P V : B fragments through transposing loads of the V tile
    {
        const int mi = lane >> 3, r8 = lane & 7;
        const int row = kb * 16 + (mi & 1) * 8 + r8;
#pragma unroll
        for (int n2 = 0; n2 < DH / 16; ++n2) {
            const int cfull = n2 * 2 + (mi >> 1);
            const uint32_t addr = vt + (cfull >> 3) * HALF_BYTES + row * 128 +
                                  ((((cfull & 7) ^ (row & 7))) << 4);
            uint32_t b[4];
            ptx::ldmatrix_x4_trans(b, addr);
            b[0] &= vm0; b[1] &= vm1; b[2] &= vm0; b[3] &= vm1;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                float(&acc)[4] = o[n2 * 2 + t];
                acc[0] *= corr[0]; acc[1] *= corr[0];
                if (hi_rows) { acc[2] *= corr[1]; acc[3] *= corr[1]; }
                ptx::mma_bf16_16816(acc, pa, b[2 * t], b[2 * t + 1]);
            }
        }
    }
}

template <int DH>
__global__ void __launch_bounds__(THREADS, 2)
shared_prefix_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_ks,
                     const __grid_constant__ CUtensorMap tm_vs) {
    using T = Tile<DH>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t bars = base + T::STAGES * T::STAGE_BYTES;        // full[s] at +16s, empty[s] at +16s+8
    volatile int *dead = reinterpret_cast<volatile int *>(gen_base + T::STAGES * T::STAGE_BYTES + 128);
    int *sid = reinterpret_cast<int *>(gen_base + T::STAGES * T::STAGE_BYTES + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int G = p.Hq / p.Hkv;
    const int parts = p.splits_sh;

    if (threadIdx.x == 0) {
        for (int s = 0; s < T::STAGES; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, NW);
        }
        *dead = 0;
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_ks); ptx::prefetch_tmap(&tm_vs);
    }

    const int part = blockIdx.x % p.splits_sh;
    const int h = (blockIdx.x / p.splits_sh) % p.Hkv;
    const int unit0 = (blockIdx.x / (p.splits_sh * p.Hkv)) * p.upc;      // first unit of the group
    const int upw = 16 / G;                 // units per warp

    // shared-segment id of every unit of the group: >= 0 valid, -1 none / out of range / bad
    for (int j = threadIdx.x; j < p.upc; j += THREADS) {
        const int i = unit0 + j;
        int s = -1;
        if (i < p.n_q) {
            s = p.sh_id[i];
            if (s >= p.n_shared || s < 0) s = -1;
        }
        sid[j] = s;
    }
    __syncthreads();

    // ---- per-thread state of the consumer warps
    uint32_t qa[DH / 16][4];
    float o[DH / 8][4];
    float m[2] = {-CUDART_INF_F, -CUDART_INF_F}, l[2] = {0.f, 0.f};
    int row_unit[2] = {-1, -1};             // query index of rows g and g+8 (-1: padding row)
    int row_head[2] = {0, 0};
    if (warp < NW) {
#pragma unroll
        for (int rs = 0; rs < 2; ++rs) {
            const int r = g + 8 * rs;
            if (r < upw * G) {
                const int i = unit0 + warp * upw + r / G;
                if (i < p.n_q) { row_unit[rs] = i; row_head[rs] = h * G + r % G; }
            }
        }
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int rs = e & 1;                         // a0,a2: row g ; a1,a3: row g+8
                const int col = ks * 16 + 2 * c + (e >> 1) * 8;
                uint32_t v = 0u;
                if (row_unit[rs] >= 0)
                    v = *reinterpret_cast<const uint32_t *>(
                        p.q + ((size_t)row_unit[rs] * p.Hq + row_head[rs]) * DH + col);
                qa[ks][e] = v;
            }
#pragma unroll
        for (int nt = 0; nt < DH / 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
    }

    int tg = 0;                               // tiles issued / consumed so far (ring position)

    // One pass streams rows [r0, r1) of one (segment, kv head) through the ring.
    auto run_pass = [&](const CUtensorMap *mk, const CUtensorMap *mv, long long row_base, int r0, int r1,
                        bool act0, bool act1) {
        const int ntiles = (r1 - r0 + BN - 1) / BN;
        if (warp == NW) {
            if (lane == 0) {
                for (int t = 0; t < ntiles; ++t) {
                    const int it = tg + t, s = it % T::STAGES;
                    if (*dead) break;
                    if (!ptx::mbar_wait(bars + 16 * s + 8, ((it / T::STAGES) & 1) ^ 1)) {
                        *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT); break;
                    }
                    const uint32_t full = bars + 16 * s;
                    const uint32_t kd = base + s * T::STAGE_BYTES, vd = kd + T::TILE_BYTES;
                    const int y = (int)(row_base + r0 + (long long)t * BN);
                    ptx::mbar_arrive_expect_tx(full, T::STAGE_BYTES);
#pragma unroll
                    for (int hh = 0; hh < T::HALVES; ++hh) {
                        ptx::tma_load_2d(kd + hh * HALF_BYTES, mk, hh * 64, y, full);
                        ptx::tma_load_2d(vd + hh * HALF_BYTES, mv, hh * 64, y, full);
                    }
                }
            }
        } else {
            for (int t = 0; t < ntiles; ++t) {
                const int it = tg + t, s = it % T::STAGES;
                if (*dead) break;
                if (!ptx::mbar_wait(bars + 16 * s, (it / T::STAGES) & 1)) {
                    *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT); break;
                }
                const uint32_t kt = base + s * T::STAGE_BYTES, vt = kt + T::TILE_BYTES;
                const int nvalid = min(BN, (r1 - r0) - t * BN);
                for (int kb = 0; kb * 16 < nvalid; ++kb)
                    process_block<DH>(kt, vt, kb, min(16, nvalid - kb * 16), qa, o, m, l, p.scale_log2, lane,
                                      act0, act1, true);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bars + 16 * s + 8);
            }
        }
        tg += ntiles;
    };

    {
        // ---- shared prefix: one pass per distinct segment id present in the group
        int last = -1;
        for (;;) {
            int cur = 0x7FFFFFFF;
            for (int j = 0; j < p.upc; ++j) {
                const int s = sid[j];
                if (s > last && s < cur) cur = s;
            }
            if (cur == 0x7FFFFFFF) break;
            last = cur;
            int r0, r1;
            part_range(max(0, min(p.sh_len[cur], p.cap_sh)), p.splits_sh, part, r0, r1);
            bool a0 = false, a1 = false;
            if (warp < NW) {
                const int j0 = warp * upw + g / G, j1 = warp * upw + (g + 8) / G;
                a0 = row_unit[0] >= 0 && sid[j0] == cur;
                a1 = row_unit[1] >= 0 && sid[j1] == cur;
            }
            run_pass(&tm_ks, &tm_vs, ((long long)cur * p.Hkv + h) * p.cap_sh, r0, r1, a0, a1);
        }
        if (warp < NW) {
#pragma unroll
            for (int rs = 0; rs < 2; ++rs) {
                l[rs] += __shfl_xor_sync(0xffffffffu, l[rs], 1);
                l[rs] += __shfl_xor_sync(0xffffffffu, l[rs], 2);
                if (row_unit[rs] < 0) continue;
                const size_t qh = (size_t)row_unit[rs] * p.Hq + row_head[rs];
                float *dst = p.partials + (qh * parts + part) * (DH + 2);
#pragma unroll
                for (int nt = 0; nt < DH / 8; ++nt)
                    *reinterpret_cast<float2 *>(dst + nt * 8 + 2 * c) =
                        make_float2(o[nt][2 * rs], o[nt][2 * rs + 1]);
                if (c == 0) { dst[DH] = m[rs]; dst[DH + 1] = l[rs]; }
            }
        }
    }
}

template <int DH>
cudaError_t run(photon_ctx *ctx, AttnParams p, cudaStream_t st, long long *launches) {
    using T = Tile<DH>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(shared_prefix_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             T::SMEM);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const int G = p.Hq / p.Hkv;
    p.upc = NW * (16 / G);
    const int groups = (p.n_q + p.upc - 1) / p.upc;
    const CUtensorMap *t;
    CUtensorMap mks, mvs;
    if (!(t = ctx->tmaps.get(p.ks, (uint64_t)p.n_shared * p.Hkv * p.cap_sh, DH, BN))) return cudaErrorInvalidValue;
    mks = *t;
    if (!(t = ctx->tmaps.get(p.vs, (uint64_t)p.n_shared * p.Hkv * p.cap_sh, DH, BN))) return cudaErrorInvalidValue;
    mvs = *t;
    shared_prefix_kernel<DH><<<groups * p.Hkv * p.splits_sh, THREADS, T::SMEM, st>>>(p, mks, mvs);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_shared_prefix_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                                           long long *launches) {
    return p.dh == 64 ? run<64>(ctx, p, st, launches) : run<128>(ctx, p, st, launches);
}
