// Two small kernels that measure or exercise the machinery the attention kernels
// are built on; neither takes part in a decode step.
//
// Read-ceiling probe: how fast can `bytes` of device memory be brought into
// shared memory by a kernel shaped like the attention kernels, when nothing is
// computed?  Same launch (programmatic dependent launch behind the call before
// it), same kind of grid (persistent, up to two CTAs per SM), same ring (three
// stages of two 16 KiB bulk copies, one thread issuing, mbarriers both ways).
// The consumer only adds up one 32-bit word of every 128 bytes it was given, so
// that the copies cannot be dropped and a test can check that every byte
// arrived.  The time of this kernel on a buffer of the size an attention call
// reads is the ceiling that call is measured against beside the HBM peak: at
// tens of megabytes a read is bound by start-up and drain, not by bandwidth.
#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

namespace {

constexpr int PIECE = 16 * 1024;            // one bulk copy
constexpr int CHUNK = 2 * PIECE;            // one ring stage (a K tile and a V tile of the attention kernel)
constexpr int P_STAGES = 3;
constexpr int P_THREADS = 64;               // warp 0: one thread issues the copies; warp 1 consumes

__global__ void __launch_bounds__(P_THREADS, 2)
read_probe_kernel(const uint8_t *src, long long n_chunks, int tail_bytes, unsigned int *sum_out, int32_t *status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = ptx::smem_u32(smem);
    const uint32_t bars = base + P_STAGES * CHUNK;              // full[s] at +16s, empty[s] at +16s+8
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) {
            ptx::mbar_init(bars + 16 * s, 1);
            ptx::mbar_init(bars + 16 * s + 8, 1);
        }
        ptx::mbar_fence_init();
    }
    __syncthreads();
    ptx::grid_dep_launch();
    ptx::grid_dep_wait();
    // chunks [c0, c1) of the buffer; the last chunk of the buffer may be short (tail_bytes, a multiple of 16)
    const long long total = n_chunks + (tail_bytes ? 1 : 0);
    const long long c0 = total * blockIdx.x / gridDim.x, c1 = total * (blockIdx.x + 1) / gridDim.x;
    const int n = (int)(c1 - c0);
    auto bytes_of = [&](long long c) { return c < n_chunks ? CHUNK : tail_bytes; };
    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < n; ++it) {
                const int s = it % P_STAGES;
                if (it >= P_STAGES && !ptx::mbar_wait(bars + 16 * s + 8, ((it / P_STAGES) & 1) ^ 1)) {
                    atomicOr(status, PHOTON_DEV_TIMEOUT);
                    break;
                }
                const int b = bytes_of(c0 + it);
                const uint8_t *g = src + (size_t)(c0 + it) * CHUNK;
                ptx::mbar_arrive_expect_tx(bars + 16 * s, b);
                const int first = min(b, PIECE);
                ptx::bulk_load(base + s * CHUNK, g, first, bars + 16 * s);
                if (b > first) ptx::bulk_load(base + s * CHUNK + PIECE, g + PIECE, b - first, bars + 16 * s);
            }
        }
        return;
    }
    unsigned int sum = 0;
    for (int it = 0; it < n; ++it) {
        const int s = it % P_STAGES;
        if (!ptx::mbar_wait(bars + 16 * s, (it / P_STAGES) & 1)) {
            if (lane == 0) atomicOr(status, PHOTON_DEV_TIMEOUT);
            break;
        }
        const int b = bytes_of(c0 + it);
        for (int off = lane * 128; off < b; off += 32 * 128) sum += ptx::lds32(base + s * CHUNK + off);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bars + 16 * s + 8);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0 && sum_out) atomicAdd(sum_out, sum);
}

// Wait probe: one thread waits, with a short limit, on an mbarrier that nobody arrives at.  The wait gives
// up, the kernel sets PHOTON_DEV_TIMEOUT, bumps a ticket (as a kernel that stopped half way would leave
// one behind) and returns by itself: the path every bounded wait of the library takes when it runs out.
__global__ void wait_probe_kernel(unsigned long long limit_ns, int32_t *status, int32_t *ticket) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = ptx::smem_u32(&bar);
    ptx::mbar_init(b, 1);
    ptx::mbar_fence_init();
    if (!ptx::mbar_wait(b, 0, limit_ns)) {
        atomicOr(status, PHOTON_DEV_TIMEOUT);
        if (ticket) atomicAdd(ticket, 1);
    }
}

}  // namespace

cudaError_t launch_wait_probe(photon_ctx *ctx, unsigned long long limit_ns, cudaStream_t st, long long *launches) {
    wait_probe_kernel<<<1, 1, 0, st>>>(limit_ns, ctx->status, ctx->tickets);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_read_probe(photon_ctx *ctx, const void *src, size_t bytes, int ctas, unsigned int *sum_out,
                              cudaStream_t st, long long *launches) {
    if (bytes == 0) return cudaSuccess;
    constexpr size_t smem = (size_t)P_STAGES * CHUNK + 64;
    static size_t smem_set[kMaxDevices] = {};
    if (const cudaError_t e = ensure_dynamic_smem(read_probe_kernel, smem, ctx->device, smem_set)) return e;
    const long long n_chunks = (long long)(bytes / CHUNK);
    const int tail = (int)(bytes % CHUNK);
    const long long total = n_chunks + (tail ? 1 : 0);
    int grid = ctas > 0 ? std::min(ctas, ctx->max_ctas) : coarse_attn_grid(ctx->max_ctas, total);
    grid = (int)std::max<long long>(1, std::min<long long>(grid, total));
    const cudaError_t e = launch_dependent(read_probe_kernel, dim3(grid), dim3(P_THREADS), smem, st, 0,
                                           static_cast<const uint8_t *>(src), n_chunks, tail, sum_out, ctx->status);
    ++*launches;
    return e != cudaSuccess ? e : cudaGetLastError();
}
