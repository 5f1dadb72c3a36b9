// Context converter U^(l) (Section 2.1.2): U[b, n] = sum_k x[b,k] W[k,n] (+ bias[n]),
// n = r*D + j for prefix r, feature j.
//
// A dense contraction on the 5th-generation tensor cores.  A CTA owns a
// [128 batch rows x NT output columns] tile of U: the batch rows are the M
// side, a slab of NT weight columns is the N side, and the accumulator lives
// in TMEM.  Only as many x rows as the batch needs (rounded up to 16, 32, 64 or
// 128) are fetched per K block; the MMA still spans 128 rows, and the rows it
// reads beyond the fetched ones are whatever shared memory holds: they only
// reach accumulator rows that are never read back.  A smaller x box makes a
// stage smaller, so a small batch gets a deeper ring of weight tiles in flight.
// One warp feeds a ring of TMA loads (x atoms and weight atoms for 128 K
// elements per stage), one warp issues tcgen05.mma on the swizzled atoms (in both
// an elected lane does the issuing), four warps read the accumulator back with
// tcgen05.ld, add the bias, round once to bf16 and store.  Every weight element leaves HBM exactly once; at small batch the
// kernel is bound by that stream, at large batch by the tensor pipe.
//
// The same kernel serves any y = x W + b with K and N multiples of 64 (the
// context chunker's linear map, Section 2.1.1: K = C_L * D, N = D).  When N is
// so small that the output tiles would leave most SMs without a share of the
// weight stream, the K range of a tile is split over the CTAs of a thread-block
// cluster: each accumulates its slice, the others stage their fp32 tile in
// their (by then free) ring and send it to the first CTA's ring with one bulk
// copy through distributed shared memory; that CTA adds the tiles in rank order,
// so the result does not depend on timing.
#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int BM = 128;                 // batch rows per CTA (UMMA M)
constexpr int BK = 64;                  // K elements per swizzle atom (one 128-byte row)
template <int NT> __host__ __device__ constexpr int atoms_per_stage() { return NT >= 256 ? 1 : 2; }   // 128 (64) K elements per barrier round trip
constexpr int CONV_THREADS = 224;       // warp 0: TMA, warps 1 and 6: MMA (1 owns TMEM), warps 2-5: epilogue
// With narrow weight slabs two warps issue MMAs: they take alternate stages and accumulate into
// separate TMEM columns, because issuing a tcgen05.mma costs one thread more time than a narrow
// MMA takes to run; the epilogue adds the accumulators.  Wide slabs gain nothing from it.
template <int NT> __host__ __device__ constexpr int mma_warps() { return NT <= 64 ? 2 : 1; }

constexpr int MAX_STAGES = 12;
constexpr int RING_BYTES = 192 * 1024;  // one CTA per SM; more output tiles than SMs run as further waves

template <int NT>
struct ConvTile {
    static constexpr int B_BYTES = NT * BK * 2;           // weight atom: 8 / 16 KiB
    // slack after the ring: the MMA reads 128 rows from every x atom, also past a short x box
    static constexpr int extra = BM * BK * 2 + 1024 + 512;
};

__host__ __device__ inline int conv_stages(int ring_bytes, int a_bytes, int b_bytes, int ka) {
    const int s = ring_bytes / (ka * (a_bytes + b_bytes));
    return s < MAX_STAGES ? s : MAX_STAGES;
}

// The loops of the TMA warp and of the MMA warp are run by the whole warp (so that their
// address arithmetic stays warp-uniform); one elected lane issues the asynchronous operations.
// GATED (slabs of 128 columns only): the gate/up projection of the MLP with its activation folded in.  W is
// [gate | up] with N = 2F columns; a CTA takes 64 gate columns and the 64 up columns of the same features, and
// writes silu(gate) * up for them into U [B, F] (both projections rounded to bf16 first, as when they are
// stored and read back by the activation kernel).  No bias, no residual, no split of K.
template <int NT, bool W_IN_MAJOR, bool SPLIT, bool GATED = false>
__global__ void __launch_bounds__(CONV_THREADS, 1)
converter_umma_kernel(const ConvParams p, const __grid_constant__ CUtensorMap tm_x,
                      const __grid_constant__ CUtensorMap tm_w) {
    using T = ConvTile<NT>;
    constexpr int KA = atoms_per_stage<NT>();
    constexpr int RING = RING_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - ptx::smem_u32(smem_raw));
    const int a_bytes = p.x_rows * BK * 2;                       // x atom of this launch
    const int stage_bytes = KA * (a_bytes + T::B_BYTES);         // [x atoms][weight atoms]
    const int n_stages = conv_stages(RING, a_bytes, T::B_BYTES, KA);
    constexpr int TAIL = RING + BM * BK * 2;
    const uint32_t bars = base + TAIL;                           // full[s] +16s, empty[s] +16s+8
    const uint32_t bar_acc = bars + 16 * MAX_STAGES;
    const uint32_t bar_rx = bar_acc + 8;                         // split K: the other CTAs' tiles have landed here
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gen + TAIL + 16 * MAX_STAGES + 16);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ks = SPLIT ? p.ksplit : 1;                         // CTAs (one cluster) that share an output tile
    const int zr = ks > 1 ? (int)(blockIdx.x % ks) : 0;          // = rank in the cluster: which slice of K
    static_assert(!GATED || (NT == 128 && !SPLIT), "the gated form takes 64 gate and 64 up columns, whole K");
    const int n0 = (int)(blockIdx.x / ks) * (GATED ? NT / 2 : NT), m0 = blockIdx.y * BM;
    const int up0 = p.N / 2 + n0;                                // GATED: first of this CTA's up columns
    constexpr int MMA_WARPS = mma_warps<NT>();
    const uint32_t stg_bytes = (uint32_t)p.x_rows * NT * 4;      // the fetched rows of one fp32 tile, stored [column][row]
    const int a_lo = (p.D / BK) * zr / ks, n_atoms = (p.D / BK) * (zr + 1) / ks - a_lo;
    const int n_steps = (n_atoms + KA - 1) / KA;

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, 1);
        }
        ptx::mbar_init(bar_acc, MMA_WARPS);
        ptx::mbar_init(bar_rx, 1);
        ptx::mbar_fence_init();
        if (ks > 1 && zr == 0) ptx::mbar_arrive_expect_tx(bar_rx, (ks - 1) * stg_bytes);
        ptx::prefetch_tmap(&tm_x); ptx::prefetch_tmap(&tm_w);
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t *>(tmem_slot)), MMA_WARPS * NT);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    ptx::grid_dep_launch();                 // one CTA per SM; the next kernel lines up once the last wave has started

    // The weights never come from the kernel before this one, x may: the ring's first turn requests its
    // weight atoms at once and its x atoms once the dependency wait has returned, so that the weight stream
    // already runs under the tail of the predecessor.  The same thread issues both, after it has told the
    // stage's barrier how many bytes to expect: were another warp to issue the x atoms, then with no
    // predecessor in flight (calls launched one by one) an x atom could land before its stage's byte count is
    // posted.  Everything else this kernel does with global memory follows from x having landed.
    auto load_x = [&](int st, int s) {
        const int atoms = min(KA, n_atoms - st * KA);
        const uint32_t a_dst = base + s * stage_bytes;
        for (int j = 0; j < atoms; ++j)
            ptx::tma_load_2d(a_dst + j * a_bytes, &tm_x, (a_lo + st * KA + j) * BK, m0, bars + 16 * s);   // x[m0.., k0..]
    };
    const int ahead = min(n_steps, n_stages);              // the ring starts empty: no stage to wait for

    if (warp == 0) {
        auto load_w = [&](int st, int s) {
            const int atoms = min(KA, n_atoms - st * KA);
            const uint32_t full = bars + 16 * s;
            const uint32_t b_dst = base + s * stage_bytes + KA * a_bytes;
            for (int j = 0; j < atoms; ++j) {
                const int k0 = (a_lo + st * KA + j) * BK;
                if (!W_IN_MAJOR) {
                    if (GATED) {                                                         // two boxes of 64 rows: gate, then up
                        ptx::tma_load_2d(b_dst + j * T::B_BYTES, &tm_w, k0, n0, full);
                        ptx::tma_load_2d(b_dst + j * T::B_BYTES + 64 * 128, &tm_w, k0, up0, full);
                    } else {
                        ptx::tma_load_2d(b_dst + j * T::B_BYTES, &tm_w, k0, n0, full);   // W[n0.., k0..]  (K-major)
                    }
                } else {
#pragma unroll
                    for (int jj = 0; jj < NT / 64; ++jj)                                 // W[k0.., n0+64jj..] (N-major)
                        ptx::tma_load_2d(b_dst + j * T::B_BYTES + jj * (BK * 128), &tm_w,
                                         GATED ? (jj == 0 ? n0 : up0) : n0 + 64 * jj, k0, full);
                }
            }
        };
        if (ptx::elect_one())
            for (int st = 0; st < ahead; ++st) {
                ptx::mbar_arrive_expect_tx(bars + 16 * st, min(KA, n_atoms - st * KA) * (a_bytes + T::B_BYTES));
                load_w(st, st);
            }
        __syncwarp();
        ptx::grid_dep_wait();               // x may be the output of the kernel before this one
        if (ptx::elect_one())
            for (int st = 0; st < ahead; ++st) load_x(st, st);
        __syncwarp();
        int s = ahead == n_stages ? 0 : ahead;
        uint32_t phase = ahead == n_stages ? 1 : 0;
        for (int st = ahead; st < n_steps; ++st) {
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(bars + 16 * s + 8, phase ^ 1))) {
                if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
                break;
            }
            if (ptx::elect_one()) {
                ptx::mbar_arrive_expect_tx(bars + 16 * s, min(KA, n_atoms - st * KA) * (a_bytes + T::B_BYTES));
                load_x(st, s);
                load_w(st, s);
            }
            __syncwarp();
            if (++s == n_stages) { s = 0; phase ^= 1; }
        }
    } else if (warp == 1 || (warp == 6 && MMA_WARPS == 2)) {
        constexpr uint32_t idesc = ptx::umma_idesc_bf16(BM, NT, false, W_IN_MAJOR);
        const int me = warp == 1 ? 0 : 1;                  // which accumulator, and which stages
        const uint32_t acc = tmem + me * NT;
        const int last_mine = n_steps - 1 >= me ? n_steps - 1 - ((n_steps - 1 - me) % MMA_WARPS) : -1;
        int s = 0;
        uint32_t phase = 0;
        bool first = true;
        if (last_mine < 0 && ptx::elect_one()) ptx::mbar_arrive(bar_acc);      // fewer steps than MMA warps
        for (int st = 0; st < n_steps; ++st) {
            if (st % MMA_WARPS != me) {
                if (++s == n_stages) { s = 0; phase ^= 1; }
                continue;
            }
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(bars + 16 * s, phase))) {
                if (lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
                break;
            }
            ptx::tc_fence_after();
            const int atoms = min(KA, n_atoms - st * KA);
            const uint32_t a_addr = base + s * stage_bytes, b_addr = a_addr + KA * a_bytes;
            if (ptx::elect_one()) {
                for (int j = 0; j < atoms; ++j) {
                    const uint64_t adesc = ptx::umma_desc_sw128(a_addr + j * a_bytes, 0, 1024);
                    const uint64_t bdesc = W_IN_MAJOR ? ptx::umma_desc_sw128(b_addr + j * T::B_BYTES, BK * 128, 1024)
                                                      : ptx::umma_desc_sw128(b_addr + j * T::B_BYTES, 0, 1024);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        // advance 16 K elements: 32 bytes inside the swizzled row (K-major),
                        // 16 rows of 128 bytes (N-major); the address field counts 16-byte units
                        const uint64_t a_k = adesc + (uint64_t)(k * 2);
                        const uint64_t b_k = bdesc + (uint64_t)(W_IN_MAJOR ? k * 128 : k * 2);
                        ptx::umma_bf16(acc, a_k, b_k, idesc, !first || (j | k) != 0);
                    }
                }
                ptx::umma_commit(bars + 16 * s + 8);       // frees the stage once these MMAs have read it
                if (st == last_mine) ptx::umma_commit(bar_acc);       // this warp's accumulator is complete
            }
            first = false;
            __syncwarp();
            if (++s == n_stages) { s = 0; phase ^= 1; }
        }
    }
    // epilogue: warp w (2..5) reads TMEM lanes [32*(w%4), +32) = batch rows m0 + that range
    const bool epi = warp >= 2 && warp <= 5;
    const int quad = warp & 3;
    bool ok = true;
    if (epi) {
        ok = ptx::mbar_wait(bar_acc, 0);
        if (!ok && lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
        ptx::tc_fence_after();
        ptx::grid_dep_wait();               // long since over; these warps read the residual and write the output
    }
    if (ks > 1) ptx::cluster_sync();        // every CTA of the cluster is done with its ring
    if (epi) {
        const int row = quad * 32 + lane, b = m0 + row;
        if (ks > 1 && zr == 0) {
            const bool got = ptx::mbar_wait(bar_rx, 0);
            if (!got && lane == 0) atomicOr(p.status, PHOTON_DEV_TIMEOUT);
            ok = ok && got;
        }
        if constexpr (GATED) {
            const int F = p.N / 2;
#pragma unroll 1
            for (int c0 = 0; c0 < NT / 2; c0 += 32) {
                uint32_t g[32], u[32];
                ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + c0, g);
                ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + NT / 2 + c0, u);
                ptx::tmem_ld_wait();
                if (ok && b < p.B) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.U + (size_t)b * F + n0 + c0);
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float g0 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(g[v * 8 + 2 * e])));
                            const float g1 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(g[v * 8 + 2 * e + 1])));
                            const float u0 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(u[v * 8 + 2 * e])));
                            const float u1 = __bfloat162float(__float2bfloat16_rn(__uint_as_float(u[v * 8 + 2 * e + 1])));
                            __nv_bfloat162 o = __floats2bfloat162_rn(g0 / (1.f + __expf(-g0)) * u0, g1 / (1.f + __expf(-g1)) * u1);
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
            ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + c0, r);
            ptx::tmem_ld_wait();
            if (MMA_WARPS == 2 && n_steps > 1) {           // second accumulator (untouched when there is one step)
                uint32_t r2[32];
                ptx::tmem_ld_32x32(tmem + ((uint32_t)(quad * 32) << 16) + NT + c0, r2);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) + __uint_as_float(r2[e]));
            }
            if (zr != 0) {                                 // stage this slice's tile for the first CTA
                if (row < p.x_rows) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        *reinterpret_cast<uint32_t *>(gen + ((size_t)(c0 + e) * p.x_rows + row) * 4) = r[e];
                }
                continue;
            }
            for (int z = 1; z < ks && row < p.x_rows; ++z) {   // add the other slices in rank order
                const float *part = reinterpret_cast<const float *>(gen + (size_t)(z - 1) * stg_bytes);
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    r[e] = __float_as_uint(__uint_as_float(r[e]) + part[(size_t)(c0 + e) * p.x_rows + row]);
            }
            if (ok && b < p.B) {
                uint4 *dst = reinterpret_cast<uint4 *>(p.U + (size_t)b * p.N + n0 + c0);
                const uint4 *res = p.residual ? reinterpret_cast<const uint4 *>(p.residual + (size_t)b * p.N + n0 + c0) : nullptr;
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t w[4];
                    const uint4 rv = res ? __ldcg(res + v) : make_uint4(0u, 0u, 0u, 0u);
                    const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float f0 = __uint_as_float(r[v * 8 + 2 * e]) + bf16_lo(rw[e]);
                        float f1 = __uint_as_float(r[v * 8 + 2 * e + 1]) + bf16_hi(rw[e]);
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
        }                                                  // (not GATED)
        if (zr != 0) {
            ptx::fence_proxy_async();                      // the staged tile is read by the bulk copy
            ptx::named_bar_sync(1, 128);                   // the four epilogue warps
            if (warp == 2 && ptx::elect_one())
                ptx::bulk_copy_to_peer(ptx::map_cluster(base + (uint32_t)(zr - 1) * stg_bytes, 0), base, stg_bytes,
                                       ptx::map_cluster(bar_rx, 0));
        }
    }
    if (ks > 1) ptx::cluster_sync();        // the first CTA has every tile: the senders' rings may go
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, MMA_WARPS * NT);
    }
}

template <int NT, bool IN_MAJOR, bool SPLIT, bool GATED = false>
cudaError_t run_as(photon_ctx *ctx, const ConvParams &p, const CUtensorMap &mx, const CUtensorMap &mw, dim3 grid,
                   cudaStream_t st) {
    using T = ConvTile<NT>;
    constexpr size_t smem = (size_t)RING_BYTES + T::extra;
    static size_t smem_set[kMaxDevices] = {};
    if (const cudaError_t e = ensure_dynamic_smem(converter_umma_kernel<NT, IN_MAJOR, SPLIT, GATED>, smem, ctx->device, smem_set)) return e;
    return launch_dependent(converter_umma_kernel<NT, IN_MAJOR, SPLIT, GATED>, grid, dim3(CONV_THREADS), smem, st,
                            p.ksplit > 1 ? p.ksplit : 0, p, mx, mw);
}

// out [B, F] = silu(x Wg) * (x Wu) for w = [Wg | Wu] (N = 2F columns), 64 features per CTA.
template <bool IN_MAJOR>
cudaError_t run_gated(photon_ctx *ctx, ConvParams p, cudaStream_t st, long long *launches) {
    p.x_rows = p.B > 64 ? 128 : p.B > 32 ? 64 : p.B > 16 ? 32 : 16;
    p.ksplit = 1;
    const CUtensorMap *t;
    CUtensorMap mx, mw;
    if (!(t = ctx->tmaps.get(p.x, (uint64_t)p.B, (uint64_t)p.D, p.x_rows))) return cudaErrorInvalidValue;
    mx = *t;
    // [K, N] in boxes of 64 k x 64 n, or [N, K] in boxes of 64 n x 64 k (gate rows and up rows are fetched apart)
    t = IN_MAJOR ? ctx->tmaps.get(p.w, (uint64_t)p.D, (uint64_t)p.N, BK) : ctx->tmaps.get(p.w, (uint64_t)p.N, (uint64_t)p.D, 64);
    if (!t) return cudaErrorInvalidValue;
    mw = *t;
    const dim3 grid(p.N / 128, (p.B + BM - 1) / BM);
    const cudaError_t e = run_as<128, IN_MAJOR, false, true>(ctx, p, mx, mw, grid, st);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <int NT, bool IN_MAJOR>
cudaError_t run(photon_ctx *ctx, ConvParams p, cudaStream_t st, long long *launches) {
    p.x_rows = p.B > 64 ? 128 : p.B > 32 ? 64 : p.B > 16 ? 32 : 16;
    const CUtensorMap *t;
    CUtensorMap mx, mw;
    if (!(t = ctx->tmaps.get(p.x, (uint64_t)p.B, (uint64_t)p.D, p.x_rows))) return cudaErrorInvalidValue;
    mx = *t;
    if (IN_MAJOR) t = ctx->tmaps.get(p.w, (uint64_t)p.D, (uint64_t)p.N, BK);        // [K, N], boxes of 64 k x 64 n
    else t = ctx->tmaps.get(p.w, (uint64_t)p.N, (uint64_t)p.D, NT);                 // [N, K], boxes of NT n x 64 k
    if (!t) return cudaErrorInvalidValue;
    mw = *t;
    if (p.ksplit < 1) p.ksplit = 1;
    dim3 grid(p.ksplit * (p.N / NT), (p.B + BM - 1) / BM);
    cudaError_t e;
    if constexpr (NT == 64)
        e = p.ksplit > 1 ? run_as<NT, IN_MAJOR, true>(ctx, p, mx, mw, grid, st) : run_as<NT, IN_MAJOR, false>(ctx, p, mx, mw, grid, st);
    else
        e = run_as<NT, IN_MAJOR, false>(ctx, p, mx, mw, grid, st);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// y = x W + b for any K (p.D) and N that are multiples of 64.  Few output tiles: narrow slabs, then the
// K range split over clusters of 2 or 4 CTAs, as long as a CTA keeps at least 8 K blocks of 64.
cudaError_t launch_linear(photon_ctx *ctx, ConvParams p, cudaStream_t st, long long *launches) {
    if (p.B == 0) return cudaSuccess;
    const int m_tiles = (p.B + BM - 1) / BM;
    const bool wide = p.B > 128 && p.N % 128 == 0 && (p.N / 128) * m_tiles * 2 >= ctx->sm_count;
    const bool wider = wide && p.N % 256 == 0 && (p.N / 256) * m_tiles >= 100;
    // narrow slabs that would need a second wave of CTAs: twice as wide, one wave
    const bool second_wave = !wide && p.N % 128 == 0 && (long long)(p.N / 64) * m_tiles > ctx->sm_count &&
                             (long long)(p.N / 128) * m_tiles <= ctx->sm_count;
    const int nt = wider ? 256 : (wide || second_wave) ? 128 : 64;
    p.ksplit = 1;
    if (nt == 64)
        while (p.ksplit < 4 && (p.N / nt) * m_tiles * p.ksplit * 2 <= ctx->sm_count && (p.D / BK) / (p.ksplit * 2) >= 8)
            p.ksplit *= 2;
    if (p.w_out_major)
        return nt == 256 ? run<256, false>(ctx, p, st, launches)
                         : nt == 128 ? run<128, false>(ctx, p, st, launches) : run<64, false>(ctx, p, st, launches);
    return nt == 256 ? run<256, true>(ctx, p, st, launches)
                     : nt == 128 ? run<128, true>(ctx, p, st, launches) : run<64, true>(ctx, p, st, launches);
}

// Whether the fused gate/up form serves this shape: whole slabs of 64 features, and enough of them to occupy most
// of the GPU without a split of K (below that the plain projection, which can split K, and the activation kernel).
bool gate_up_fits_small_tiles(const photon_ctx *ctx, const ConvParams &p) {
    const long long tiles = (long long)(p.N / 128) * ((p.B + BM - 1) / BM);
    return p.N % 128 == 0 && p.D % BK == 0 && tiles * 2 >= ctx->sm_count;
}

cudaError_t launch_gate_up(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    if (p.B == 0) return cudaSuccess;
    return p.w_out_major ? run_gated<false>(ctx, p, st, launches) : run_gated<true>(ctx, p, st, launches);
}

cudaError_t launch_converter(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches) {
    if (p.B == 0) return cudaSuccess;
    // wider weight slabs once the batch is large enough for the tensor pipe to matter, as long as
    // about one CTA per SM remains
    const int m_tiles = (p.B + BM - 1) / BM;
    const bool wide = p.B > 128 && p.N % 128 == 0;
    const bool wider = wide && p.N % 256 == 0 && (p.N / 256) * m_tiles >= 100;
    if (p.w_out_major)
        return wider ? run<256, false>(ctx, p, st, launches)
                     : wide ? run<128, false>(ctx, p, st, launches) : run<64, false>(ctx, p, st, launches);
    return wider ? run<256, true>(ctx, p, st, launches)
                 : wide ? run<128, true>(ctx, p, st, launches) : run<64, true>(ctx, p, st, launches);
}
