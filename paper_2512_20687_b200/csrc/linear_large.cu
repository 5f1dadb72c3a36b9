// y = x W + b (+ residual) for batches of thousands of rows (the projections and
// MLP of a decoder layer over all in-flight chunks): the same tcgen05 contraction
// as the converter kernel, arranged for the case that is bound by the tensor
// pipe instead of by the weight stream.
//
// One persistent CTA per SM walks over [128 rows x 256 columns] output tiles in
// an order that keeps one slab of weight columns hot in L2 (all row tiles of a
// slab before the next slab).  TMEM holds two accumulators of 256 columns: while
// the four epilogue warps read one back (tcgen05.ld, bias, residual, one
// rounding to bf16, 16-byte stores), the MMA warp is already filling the other
// from the TMA ring, which the producer warp keeps running across tile
// boundaries.  Shared memory: 4 stages of one K block of 64 (x atom 16 KiB,
// weight atom 32 KiB).  Every wait is bounded; a wait that gives up sets the
// status bit and a flag that makes every role leave its loops.
//
// GATED: the gate/up projection of the MLP with its activation folded in.  The
// weight is [gate | up] (N = 2F columns); a tile takes 128 gate columns and the
// 128 up columns of the same features as its two halves, and the epilogue writes
// silu(g) * u for those 128 features: out [B, F], and the [B, 2F] intermediate
// never exists.
#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int BM = 128, BK = 64, NT = 256;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = NT * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int RING = STAGES * STAGE_BYTES;
constexpr int LL_THREADS = 192;             // warp 0: TMA, warp 1: MMA (owns TMEM), warps 2-5: epilogue
constexpr int LL_SMEM = RING + 1024 + 256;

template <bool W_IN_MAJOR, bool GATED>
__global__ void __launch_bounds__(LL_THREADS, 1)
linear_tiles_kernel(const ConvParams p, const __grid_constant__ CUtensorMap tm_x,
                    const __grid_constant__ CUtensorMap tm_w) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t bars = base + RING;                          // full[s] +16s, empty[s] +16s+8
    const uint32_t acc_full = bars + 16 * STAGES, acc_empty = acc_full + 16;   // [2] each, 8 bytes apart
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen + RING + 16 * STAGES + 32);
    volatile int *dead = reinterpret_cast<volatile int *>(gen + RING + 16 * STAGES + 40);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int F = p.N / 2;                                      // GATED: features; a tile covers 128 of them
    const int m_tiles = (p.B + BM - 1) / BM, n_tiles = GATED ? F / (NT / 2) : p.N / NT;
    const int tiles = m_tiles * n_tiles, n_atoms = p.D / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(acc_full + 8 * b, 1);
            ptx::mbar_init(acc_empty + 8 * b, 4);               // one arrival per epilogue warp
        }
        *dead = 0;
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_x); ptx::prefetch_tmap(&tm_w);
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), 2 * NT);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    ptx::grid_dep_wait();                   // x may be the output of the kernel before this one
    ptx::grid_dep_launch();

    auto give_up = [&]() {
        if (lane == 0) { atomicOr(p.status, PHOTON_DEV_TIMEOUT); *dead = 1; }
    };

    if (warp == 0) {
        // ---- producer: the ring runs on across tile boundaries ----
        int s = 0;
        uint32_t phase = 0;
        for (int t = blockIdx.x; t < tiles && !*dead; t += gridDim.x) {
            const int m0 = (t % m_tiles) * BM, n0 = (t / m_tiles) * (GATED ? NT / 2 : NT);
            for (int a = 0; a < n_atoms; ++a) {
                if (!__all_sync(0xffffffffu, ptx::mbar_wait(bars + 16 * s + 8, phase ^ 1))) { give_up(); break; }
                const uint32_t full = bars + 16 * s, a_dst = base + s * STAGE_BYTES, b_dst = a_dst + A_BYTES;
                if (ptx::elect_one()) {
                    ptx::mbar_arrive_expect_tx(full, STAGE_BYTES);
                    const int k0 = a * BK;
                    ptx::tma_load_2d(a_dst, &tm_x, k0, m0, full);                        // x[m0.., k0..]
                    if (!W_IN_MAJOR) {
                        if (GATED) {                                                      // boxes of 128 rows: gate, then up
                            ptx::tma_load_2d(b_dst, &tm_w, k0, n0, full);
                            ptx::tma_load_2d(b_dst + B_BYTES / 2, &tm_w, k0, F + n0, full);
                        } else {
                            ptx::tma_load_2d(b_dst, &tm_w, k0, n0, full);                // W[n0.., k0..]  (K-major)
                        }
                    } else {
#pragma unroll
                        for (int jj = 0; jj < NT / 64; ++jj) {                            // W[k0.., n..] (N-major), 64 columns a box
                            const int col = GATED ? (jj < 2 ? n0 + 64 * jj : F + n0 + 64 * (jj - 2)) : n0 + 64 * jj;
                            ptx::tma_load_2d(b_dst + jj * (BK * 128), &tm_w, col, k0, full);
                        }
                    }
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ---- MMA: tile i of this CTA accumulates into buffer i & 1 ----
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(BM, NT, false, W_IN_MAJOR);
        int s = 0, i = 0;
        uint32_t phase = 0;
        for (int t = blockIdx.x; t < tiles && !*dead; t += gridDim.x, ++i) {
            const int buf = i & 1;
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(acc_empty + 8 * buf, ((i >> 1) & 1) ^ 1))) { give_up(); break; }
            ptx::tc_fence_after();
            const uint32_t acc = tmem + buf * NT;
            bool ok = true;
            for (int a = 0; a < n_atoms; ++a) {
                if (!__all_sync(0xffffffffu, ptx::mbar_wait(bars + 16 * s, phase))) { give_up(); ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t a_addr = base + s * STAGE_BYTES, b_addr = a_addr + A_BYTES;
                if (ptx::elect_one()) {
                    const uint64_t adesc = ptx::umma_desc_sw128(a_addr, 0, 1024);
                    const uint64_t bdesc = W_IN_MAJOR ? ptx::umma_desc_sw128(b_addr, BK * 128, 1024)
                                                      : ptx::umma_desc_sw128(b_addr, 0, 1024);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        ptx::umma_bf16(acc, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(W_IN_MAJOR ? k * 128 : k * 2),
                                       idesc, (a | k) != 0);
                    ptx::umma_commit(bars + 16 * s + 8);       // frees the stage once these MMAs have read it
                    if (a == n_atoms - 1) ptx::umma_commit(acc_full + 8 * buf);   // this tile's accumulator is complete
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; phase ^= 1; }
            }
            if (!ok) break;
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes [32*(w%4), +32) = rows of the tile ----
        const int quad = warp & 3;
        int i = 0;
        for (int t = blockIdx.x; t < tiles && !*dead; t += gridDim.x, ++i) {
            const int buf = i & 1;
            const int m0 = (t % m_tiles) * BM, n0 = (t / m_tiles) * (GATED ? NT / 2 : NT);
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(acc_full + 8 * buf, (i >> 1) & 1))) { give_up(); break; }
            ptx::tc_fence_after();
            const int b = m0 + quad * 32 + lane;
            if constexpr (GATED) {
#pragma unroll 1
                for (int c0 = 0; c0 < NT / 2; c0 += 32) {
                    uint32_t g[32], u[32];
                    ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + buf * NT + c0, g);
                    ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + buf * NT + NT / 2 + c0, u);
                    ptx::tmem_ld_wait();
                    if (b < p.B) {
                        uint4 *dst = reinterpret_cast<uint4 *>(p.U + (size_t)b * F + n0 + c0);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // the projections are rounded to bf16 first, as when they are stored and read back
                                const float g0 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(g[v * 8 + 2 * e])));
                                const float g1 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(g[v * 8 + 2 * e + 1])));
                                const float u0 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(u[v * 8 + 2 * e])));
                                const float u1 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(u[v * 8 + 2 * e + 1])));
                                __nv_bfloat162 o = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * u0,
                                                                         g1 / (1.f + __expf(-g1)) * u1);
                                w[e] = *reinterpret_cast<uint32_t *>(&o);
                            }
                            dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            } else {
#pragma unroll 1
            for (int c0 = 0; c0 < NT; c0 += 32) {
                uint32_t r[32];
                ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + buf * NT + c0, r);
                ptx::tmem_ld_wait();
                if (b < p.B) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.U + (size_t)b * p.N + n0 + c0);
                    const uint4 *res = p.residual ? reinterpret_cast<const uint4 *>(p.residual + (size_t)b * p.N + n0 + c0) : nullptr;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint32_t w[4];
                        const uint4 rv = res ? res[v] : make_uint4(0u, 0u, 0u, 0u);
                        const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float f0 = __uint_as_float(r[v * 8 + 2 * e]) + bf16_lo(rw[e]);
                            float f1 = __uint_as_float(r[v * 8 + 2 * e + 1]) + bf16_hi(rw[e]);
                            if (p.bias) {
                                f0 += __bfloat162float(p.bias[n0 + c0 + v * 8 + 2 * e]);
                                f1 += __bfloat162float(p.bias[n0 + c0 + v * 8 + 2 * e + 1]);
                            }
                            __nv_bfloat162 o = __floats2bfloat162_rn(f0, f1);
                            w[e] = *reinterpret_cast<uint32_t *>(&o);
                        }
                        dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty + 8 * buf);          // the MMA warp may overwrite this buffer
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, 2 * NT);
    }
}

template <bool IN_MAJOR, bool GATED>
cudaError_t run_large(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    static size_t smem_set[kMaxDevices] = {};
    if (const cudaError_t e = ensure_dynamic_smem(linear_tiles_kernel<IN_MAJOR, GATED>, LL_SMEM, ctx->device, smem_set)) return e;
    const CUtensorMap *t;
    CUtensorMap mx, mw;
    if (!(t = ctx->tmaps.get(p.x, (uint64_t)p.B, (uint64_t)p.D, BM))) return cudaErrorInvalidValue;
    mx = *t;
    if (IN_MAJOR) t = ctx->tmaps.get(p.w, (uint64_t)p.D, (uint64_t)p.N, BK);        // [K, N], boxes of 64 k x 64 n
    else t = ctx->tmaps.get(p.w, (uint64_t)p.N, (uint64_t)p.D, GATED ? NT / 2 : NT);   // [N, K], boxes of 256 (128) n x 64 k
    if (!t) return cudaErrorInvalidValue;
    mw = *t;
    const int tiles = ((p.B + BM - 1) / BM) * (p.N / NT);                           // (the same count when gated)
    const cudaError_t e = launch_dependent(linear_tiles_kernel<IN_MAJOR, GATED>, dim3(std::min(tiles, ctx->sm_count)),
                                           dim3(LL_THREADS), LL_SMEM, st, 0, p, mx, mw);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// For N a multiple of 256 and more than two tiles of 128 x 256 per SM.
bool linear_wants_large_tiles(const photon_ctx *ctx, const ConvParams &p) {
    return p.N % NT == 0 && (long long)((p.B + BM - 1) / BM) * (p.N / NT) > 2ll * ctx->sm_count;
}

cudaError_t launch_linear_large(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    return p.w_out_major ? run_large<false, false>(ctx, p, st, launches) : run_large<true, false>(ctx, p, st, launches);
}

// out [B, F] = silu(x Wg) * (x Wu) for w = [Wg | Wu] with N = 2F columns; for the shapes
// linear_wants_large_tiles accepts.  No bias, no residual.
cudaError_t launch_gate_up_large(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    return p.w_out_major ? run_large<false, true>(ctx, p, st, launches) : run_large<true, true>(ctx, p, st, launches);
}
