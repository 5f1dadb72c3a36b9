// photon_coarse_attn_noalloc: the coarse decode attention for callers that must
// not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// serving process whose memory pool owns every byte of the device and treats a
// foreign allocation as a bug, in a thread that must never take the allocator's
// locks or trigger its implicit synchronisation, or after start-up in a process
// that has promised a fixed footprint.  photon_create (which allocates the
// workspace of photon_coarse_attn) is unusable there.  This entry point needs
// no context: the workspace the kernel wants (partials of caches cut by a CTA
// boundary, one arrival ticket per (unit, KV head), a status word) lives in a
// file-scope device array that is part of the loaded library image, so every
// GPU that loads the library holds those few megabytes until the process exits.
//
// The array's name in host code is only a handle, not a device address; the
// address is looked up once per device with cudaGetSymbolAddress, here, in the
// file that defines the array.  That look-up happens in the first call made on
// a device, so make one call on each device before capturing a stream into a
// graph.  Every call on a device uses the same array and finds in it whatever
// the previous call left: the tickets are cleared on the caller's stream at the
// start of each call, the partials are always written before they are read.
// Two calls that overlap on one GPU (different streams, or graphs replayed side
// by side) would race on it: keep them in stream order.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int kMaxCtas = 320;                               // grid the array is sized for
constexpr int kMaxStreams = PHOTON_NOALLOC_MAX_STREAMS;     // (unit, KV head) pairs
constexpr size_t kPartialBytes = size_t(2) * kMaxCtas * 16 * (128 + 2) * sizeof(float);
constexpr size_t kTicketBytes = size_t(kMaxStreams) * sizeof(int32_t);
constexpr size_t kScratchBytes = kPartialBytes + kTicketBytes + 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct DeviceState {
    bool ready = false;
    photon_ctx ctx;                // host-side only: no device memory of its own
};
DeviceState g_state[kMaxDevices];
std::mutex g_mutex;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" photon_status photon_coarse_attn_noalloc(const photon_config *cfg, const photon_kv *cache,
                                                    const photon_bf16 *q, photon_bf16 *out, float *lse,
                                                    float scale, int32_t *dev_status, photon_stream stream) {
    if (!cfg || !cache || !cache->k || !cache->v || !cache->len) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = *cfg;
    if (c.Hq <= 0 || c.Hkv <= 0 || c.Hq % c.Hkv != 0) return PHOTON_ERR_INVALID_ARG;
    if (c.dh != 64 && c.dh != 128) return PHOTON_ERR_UNSUPPORTED;
    if (c.Hq / c.Hkv > 16) return PHOTON_ERR_UNSUPPORTED;
    if (cache->k_shared) return PHOTON_ERR_UNSUPPORTED;           // shared prefixes need the context's workspace
    if (cache->page_table) return PHOTON_ERR_INVALID_ARG;         // contiguous caches only
    if (cache->n_units < 0 || cache->cap <= 0 || cache->max_len < 0 || cache->max_len > cache->cap)
        return PHOTON_ERR_INVALID_ARG;
    if ((long long)cache->n_units * c.Hkv > kMaxStreams) return PHOTON_ERR_WORKSPACE;   // beyond the static array
    if ((uint64_t)cache->n_units * c.Hkv * cache->cap >= (1ull << 31)) return PHOTON_ERR_UNSUPPORTED;
    if (cache->n_units > 0 && (!q || !out)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(cache->k) || !aligned16(cache->v) || !aligned16(q) || !aligned16(out))
        return PHOTON_ERR_INVALID_ARG;
    if (!(scale == scale)) return PHOTON_ERR_INVALID_ARG;
    if (cache->n_units == 0) return PHOTON_OK;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PHOTON_ERR_CUDA;
    DeviceState &s = g_state[dev];
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!s.ready) {
            // once per device, with that device current: the device address of the array
            unsigned char *base = nullptr;
            if (cudaGetSymbolAddress(reinterpret_cast<void **>(&base), g_noalloc_scratch) != cudaSuccess || !base)
                return PHOTON_ERR_CUDA;
            cudaDeviceProp prop;
            if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return PHOTON_ERR_CUDA;
            if (prop.major != 10) return PHOTON_ERR_UNSUPPORTED;
            s.ctx.device = dev;
            s.ctx.sm_count = prop.multiProcessorCount;
            s.ctx.max_ctas = std::min(kMaxCtas, prop.multiProcessorCount * coarse_attn_ctas_per_sm());
            s.ctx.attn_ctas = 0;
            s.ctx.max_splits = 1;
            s.ctx.partials = nullptr;
            s.ctx.partial_floats = 0;
            s.ctx.cta_partials = reinterpret_cast<float *>(base);
            s.ctx.tickets = reinterpret_cast<int32_t *>(base + kPartialBytes);
            s.ctx.n_tickets = kMaxStreams;
            s.ctx.status = reinterpret_cast<int32_t *>(base + kPartialBytes + kTicketBytes);
            s.ctx.launches = 0;
            if (cudaMemset(s.ctx.status, 0, sizeof(int32_t)) != cudaSuccess) return PHOTON_ERR_CUDA;
            s.ready = true;
        }
        s.ctx.cfg = c;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // tickets must read zero when the kernel starts, whatever an earlier call left behind
    if (cudaMemsetAsync(s.ctx.tickets, 0, size_t(cache->n_units) * c.Hkv * sizeof(int32_t), st) != cudaSuccess)
        return PHOTON_ERR_CUDA;

    AttnParams p{};
    p.q = reinterpret_cast<const bf16 *>(q);
    p.out = reinterpret_cast<bf16 *>(out);
    p.lse = lse;
    p.k = reinterpret_cast<const bf16 *>(cache->k);
    p.v = reinterpret_cast<const bf16 *>(cache->v);
    p.len = cache->len;
    p.n_units = cache->n_units;
    p.cap = cache->cap;
    p.max_len = cache->max_len ? cache->max_len : cache->cap;
    p.n_q = cache->n_units;
    p.Hq = c.Hq; p.Hkv = c.Hkv; p.dh = c.dh;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.splits_sh = 0;
    p.partials = nullptr;
    p.cta_partials = s.ctx.cta_partials;
    p.tickets = s.ctx.tickets;
    p.status = dev_status ? dev_status : s.ctx.status;
    std::lock_guard<std::mutex> lock(g_mutex);                 // the tensor-map cache is host state
    const cudaError_t e = launch_attention(&s.ctx, p, st, &s.ctx.launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}
