// Context converter U^(l) (Section 2.1.2): U[b, n] = sum_k x[b,k] W[k,n] (+ bias[n]),
// n = r*D + j for prefix r, feature j.
//
// A dense contraction on the 5th-generation tensor cores.  A CTA owns a
// [128 batch rows x NT output columns] tile of U: the batch rows are the M
// side (rows past the batch are zero-filled by TMA and cost no bandwidth), a
// slab of NT weight columns is the N side, and the accumulator lives in TMEM.
// One thread feeds a ring of TMA loads (x tile and weight tile per 64-wide K
// block), one thread issues tcgen05.mma on the swizzled tiles, four warps read
// the accumulator back with tcgen05.ld, add the bias, round once to bf16 and
// store.  Every weight element leaves HBM exactly once; at small batch the
// kernel is bound by that stream, at large batch by the tensor pipe.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int BM = 128;                 // batch rows per CTA (UMMA M)
constexpr int BK = 64;                  // K elements per stage (one 128-byte swizzle row)
constexpr int CONV_THREADS = 192;       // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue

template <int NT>
struct ConvTile {
    static constexpr int A_BYTES = BM * BK * 2;           // 16 KiB
    static constexpr int B_BYTES = NT * BK * 2;           // 8 / 16 KiB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = NT == 64 ? 8 : 6;       // 192 KiB of tiles either way
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 + 256;
};

template <int NT, bool W_IN_MAJOR>
__global__ void __launch_bounds__(CONV_THREADS, 1)
converter_umma_kernel(const ConvParams p, const __grid_constant__ CUtensorMap tm_x,
                      const __grid_constant__ CUtensorMap tm_w) {
    using T = ConvTile<NT>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t bars = base + T::STAGES * T::STAGE_BYTES;     // full[s] +16s, empty[s] +16s+8
    const uint32_t bar_acc = bars + 16 * T::STAGES;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen + T::STAGES * T::STAGE_BYTES + 16 * T::STAGES + 16);
    volatile int *dead = reinterpret_cast<volatile int *>(gen + T::STAGES * T::STAGE_BYTES + 16 * T::STAGES + 32);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * NT, m0 = blockIdx.y * BM;
    const int nkb = p.D / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < T::STAGES; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, 1);
        }
        ptx::mbar_init(bar_acc, 1);
        *dead = 0;
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_x); ptx::prefetch_tmap(&tm_w);
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), NT);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % T::STAGES;
                if (*dead) break;
                if (!ptx::mbar_wait(bars + 16 * s + 8, ((kb / T::STAGES) & 1) ^ 1)) {
                    *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT); break;
                }
                const uint32_t full = bars + 16 * s;
                const uint32_t a_dst = base + s * T::STAGE_BYTES, b_dst = a_dst + T::A_BYTES;
                ptx::mbar_arrive_expect_tx(full, T::STAGE_BYTES);
                ptx::tma_load_2d(a_dst, &tm_x, kb * BK, m0, full);               // x[m0.., k..]
                if (!W_IN_MAJOR) {
                    ptx::tma_load_2d(b_dst, &tm_w, kb * BK, n0, full);           // W[n0.., k..]  (K-major)
                } else {
#pragma unroll
                    for (int j = 0; j < NT / 64; ++j)                            // W[k.., n0+64j..] (N-major)
                        ptx::tma_load_2d(b_dst + j * (BK * 128), &tm_w, n0 + 64 * j, kb * BK, full);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(BM, NT, false, W_IN_MAJOR);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % T::STAGES;
                if (*dead || !ptx::mbar_wait(bars + 16 * s, (kb / T::STAGES) & 1)) {
                    if (!*dead) { *dead = 1; atomicOr(p.status, PHOTON_DEV_TIMEOUT); }
                    ok = false; break;
                }
                ptx::tc_fence_after();
                const uint32_t a_addr = base + s * T::STAGE_BYTES, b_addr = a_addr + T::A_BYTES;
                const uint64_t adesc = ptx::umma_desc_sw128(a_addr, 0, 1024);
                const uint64_t bdesc = W_IN_MAJOR ? ptx::umma_desc_sw128(b_addr, BK * 128, 1024)
                                                  : ptx::umma_desc_sw128(b_addr, 0, 1024);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    // advance 16 K elements: 32 bytes inside the swizzled row (K-major),
                    // 16 rows of 128 bytes (N-major); the address field counts 16-byte units
                    const uint64_t a_k = adesc + (uint64_t)(k * 2);
                    const uint64_t b_k = bdesc + (uint64_t)(W_IN_MAJOR ? k * 128 : k * 2);
                    ptx::umma_bf16(tmem, a_k, b_k, idesc, (kb | k) != 0);
                }
                ptx::umma_commit(bars + 16 * s + 8);       // frees the stage once these MMAs have read it
            }
            ptx::umma_commit(bar_acc);                     // accumulator complete
        }
    } else {
        // epilogue: warp w reads TMEM lanes [32*(w%4), +32) = batch rows m0 + that range
        const int quad = warp & 3;
        const int b = m0 + quad * 32 + lane;
        bool ok = !*dead && ptx::mbar_wait(bar_acc, 0);
        if (!ok && lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
        ptx::tc_fence_after();
#pragma unroll 1
        for (int c0 = 0; c0 < NT; c0 += 32) {
            uint32_t r[32];
            ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + c0, r);
            ptx::tmem_ld_wait();
            if (ok && b < p.B) {
                uint4 *dst = reinterpret_cast<uint4 *>(p.U + (size_t)b * p.N + n0 + c0);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float f0 = __uint_as_float(r[v * 8 + 2 * e]), f1 = __uint_as_float(r[v * 8 + 2 * e + 1]);
                        if (p.bias) {
                            f0 += __bfloat162float(p.bias[n0 + c0 + v * 8 + 2 * e]);
                            f1 += __bfloat162float(p.bias[n0 + c0 + v * 8 + 2 * e + 1]);
                        }
                        __nv_bfloat162 t = __floats2bfloat162_rn(f0, f1);
                        w[e] = *reinterpret_cast<uint32_t *>(&t);
                    }
                    dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, NT);
    }
}

template <int NT, bool IN_MAJOR>
cudaError_t run(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    using T = ConvTile<NT>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(converter_umma_kernel<NT, IN_MAJOR>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const CUtensorMap *t;
    CUtensorMap mx, mw;
    if (!(t = ctx->tmaps.get(p.x, (uint64_t)p.B, (uint64_t)p.D, BM))) return cudaErrorInvalidValue;
    mx = *t;
    if (IN_MAJOR) t = ctx->tmaps.get(p.w, (uint64_t)p.D, (uint64_t)p.N, BK);        // [K, N], boxes of 64 k x 64 n
    else t = ctx->tmaps.get(p.w, (uint64_t)p.N, (uint64_t)p.D, NT);                 // [N, K], boxes of NT n x 64 k
    if (!t) return cudaErrorInvalidValue;
    mw = *t;
    dim3 grid(p.N / NT, (p.B + BM - 1) / BM);
    converter_umma_kernel<NT, IN_MAJOR><<<grid, CONV_THREADS, T::SMEM, st>>>(p, mx, mw);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_converter(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    if (p.B == 0) return cudaSuccess;
    // wider weight slabs once the batch is large enough for the tensor pipe to matter
    const bool wide = p.B > 128 && p.N % 128 == 0;
    if (p.w_out_major)
        return wide ? run<128, false>(ctx, p, st, launches) : run<64, false>(ctx, p, st, launches);
    return wide ? run<128, true>(ctx, p, st, launches) : run<64, true>(ctx, p, st, launches);
}
