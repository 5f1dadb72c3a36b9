// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "photon.h"

typedef __nv_bfloat16 bf16;

// Tensor maps keyed by (base pointer, shape); entries are copied out by value.
struct TmapCache {
    static constexpr int kEntries = 64;
    struct Entry {
        const void *base;
        uint64_t rows, cols;
        uint32_t box_rows;
        CUtensorMap map;
    };
    Entry e[kEntries];
    int n = 0, next = 0;
    const CUtensorMap *get(const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
};
bool make_tmap_bf16_rows(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows);

struct photon_ctx {
    photon_config cfg;
    int device;
    int sm_count;
    int max_splits;          // resolved upper bound on key ranges per query
    float *partials;         // shared-prefix partials: [max_queries * Hq][dh + 2] floats (acc, m, l)
    size_t partial_floats;
    float *cta_partials;     // partials of streams cut by a CTA boundary: [2 * max_ctas][16][dh + 2] floats
    int max_ctas;            // most CTAs the persistent attention kernel can hold: two per SM
    int attn_ctas;           // the caller's cap on that grid (photon_set_attention_ctas), 0: the launcher chooses
    int32_t *tickets;        // one arrival counter per (unit, kv head); zero between calls
    size_t n_tickets;
    int32_t *status;         // device status word
    int32_t *work;           // two counters of the whole-chunk attention's item hand-out; zero between calls
    int32_t *readers;        // arrival counter of an attention with the append folded in; zero between calls
    long long launches;
    cudaStream_t side;       // lowest-priority stream for the chunk attention of a decode step
    cudaEvent_t ev_fork, ev_join;
    long long host_pause_ns; // photon_decode_step_host: pause between the first host-to-device copy and the first launch
    long long host_poll_us;  // photon_decode_step_host: how long the call polls the stream before it blocks on it
    cudaStream_t copy;       // carries the coarse results to the host beside the converter (photon_decode_step_host)
    cudaEvent_t ev_mid, ev_copy;
    TmapCache tmaps;
};

// Everything an attention launch needs.  A "query" i uses cache unit
// u = slot ? slot[i] : i.  Its keys are the shared segment's rows (if any)
// followed by the unit's own rows; the shared part is cut into splits_sh key
// ranges and the own part into splits_own.
struct AttnParams {
    const bf16 *q;
    bf16 *out;
    float *lse;
    const bf16 *k, *v;
    const int32_t *len;
    int n_units, cap;
    int max_len;             // host-side bound on len[] (sizes the grid)
    const bf16 *ks, *vs;
    const int32_t *sh_len, *sh_id;
    int n_shared, cap_sh;
    const int32_t *slot;
    const int32_t *page_table;   // paged cache: [n_units, pages_per_unit] page ids, or NULL
    int page_rows, pages_per_unit, n_pages;
    int n_q, Hq, Hkv, dh;
    int splits_sh;           // key ranges of a shared prefix = cluster size of its kernel (0: no shared prefix)
    int upc;                 // filled by the launcher: units per CTA on shared keys
    int own_rows;            // filled by the launcher: the units' own keys (at most this many rows each) are read by the
                             // shared-prefix kernel, which then writes the final result; 0: a second kernel reads them
    float scale_log2;        // scale * log2(e): logits are kept in the base-2 domain
    float *partials;
    float *cta_partials;
    int32_t *tickets;
    int32_t *status;
    // The step's append folded into the attention over the unit's own keys (all NULL otherwise): one new row per unit,
    // k_new, v_new [n_units, Hkv, dh], installed at row len[u] of a contiguous cache (k_w, v_w: the cache, writable),
    // len_w[u] += 1 by the last CTA to arrive on `readers` (a counter that is zero between calls).
    const bf16 *k_new, *v_new;
    bf16 *k_w, *v_w;
    int32_t *len_w;
    int32_t *readers;
};

// Whole-chunk causal attention: query t of item i (q, out: [n, R, Hq, dh]) stands at row row0 + t of
// chunk buffer u = slot ? slot[i] : i and sees rows 0 .. row0 + t of it.
struct CausalParams {
    const bf16 *q;
    bf16 *out;
    const bf16 *k, *v;
    const int32_t *len;
    const int32_t *slot;
    int n_units, cap;
    int n, R, row0;
    int gsplit;              // filled by the launcher: warps that share a (chunk, KV head), 1 or Hq / Hkv
    int32_t *work;           // filled by the launcher: {items handed out, CTAs that have finished}; zero between calls
    int Hq, Hkv, dh;
    float scale_log2;
    int32_t *status;
};

struct ConvParams {
    const bf16 *x, *w, *bias;
    const bf16 *residual;    // [B, N] added before the output is rounded, or NULL
    bf16 *U;
    int B, D, N;             // N = P * D
    int w_out_major;
    int x_rows;              // filled by the launcher: x rows fetched per K block (16, 32, 64 or 128)
    int ksplit;              // CTAs (one cluster) sharing an output tile, each on a slice of K; 0 or 1: none
    int32_t *status;
};

// Raises a kernel's dynamic shared-memory limit once per device (the attribute is per device and per
// function); `set` is the launcher's record of what each device already has.
constexpr int kMaxDevices = 64;
template <typename K>
inline cudaError_t ensure_dynamic_smem(K kernel, size_t bytes, int device, size_t (&set)[kMaxDevices]) {
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (bytes <= set[device]) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) set[device] = bytes;
    return e;
}

// Launch with programmatic stream serialization (and, optionally, a cluster width): the kernel's launch
// latency and its set-up before grid_dep_wait() overlap the tail of the kernel before it in the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    int cluster_x, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// launchers: enqueue on `st`, add the number of kernels launched to *launches,
// return the launch error (cudaSuccess when fine)
struct Paging {              // of a paged cache; table == nullptr: contiguous
    const int32_t *table;
    int page_rows, pages_per_unit, n_pages;
};
cudaError_t launch_kv_append(bf16 *k, bf16 *v, int32_t *len, int n_units, int Hkv, int cap, int dh,
                             const bf16 *k_new, const bf16 *v_new, const int32_t *unit_ids, int n,
                             int n_rows, Paging pg, int32_t *status, cudaStream_t st, long long *launches);
cudaError_t launch_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                             long long *launches);
cudaError_t launch_shared_prefix_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                                           long long *launches);
int coarse_attn_ctas_per_sm();
int coarse_attn_fold_limit();     // largest batch for which the step's append can be folded into the attention
int coarse_attn_grid(int resident_ctas, long long n_streams);
int shared_prefix_units_per_cta(int G);
int shared_prefix_own_rows();
// Whether an attention call on this cache is one launch: a shared prefix, and own caches short enough (by the caller's
// max_len) for their keys to ride along in the shared-prefix kernel.
inline bool own_keys_ride_with_prefix(const photon_kv *c) {
    return c->k_shared && !c->page_table && (c->max_len ? c->max_len : c->cap) <= shared_prefix_own_rows();
}
cudaError_t launch_chunk_attention(photon_ctx *ctx, const AttnParams &p, cudaStream_t st,
                                   long long *launches);
cudaError_t launch_chunk_causal_attention(photon_ctx *ctx, const CausalParams &p, cudaStream_t st,
                                          long long *launches);
cudaError_t launch_linear(photon_ctx *ctx, ConvParams p, cudaStream_t st, long long *launches);
bool linear_wants_large_tiles(const photon_ctx *ctx, const ConvParams &p);
cudaError_t launch_linear_large(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches);
cudaError_t launch_gate_up_large(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches);
bool gate_up_fits_small_tiles(const photon_ctx *ctx, const ConvParams &p);
cudaError_t launch_gate_up(photon_ctx *ctx, const ConvParams &p, cudaStream_t st, long long *launches);
cudaError_t launch_rmsnorm(const bf16 *x, const bf16 *gamma, float eps, bf16 *out, int rows, int cols,
                           cudaStream_t st, long long *launches);
cudaError_t launch_rope_split(const bf16 *qkv, const int32_t *pos, int period, int n, int Hq, int Hkv, int dh,
                              float theta, bf16 *q, bf16 *k, bf16 *v, cudaStream_t st, long long *launches);
// the same split with k and v written into row len[i] of unit i of a cache (contiguous or paged) and len[i] += 1
cudaError_t launch_rope_split_append(const bf16 *qkv, int n, int Hq, int Hkv, int dh, float theta, bf16 *q, bf16 *k_cache,
                                     bf16 *v_cache, int32_t *len, int cap, Paging pg, int32_t *status, cudaStream_t st,
                                     long long *launches);
cudaError_t launch_swiglu(const bf16 *gu, bf16 *out, int n, int F, cudaStream_t st, long long *launches);
cudaError_t launch_converter(photon_ctx *ctx, const ConvParams &p, cudaStream_t st,
                             long long *launches);
cudaError_t launch_read_probe(photon_ctx *ctx, const void *src, size_t bytes, int ctas, unsigned int *sum_out,
                              cudaStream_t st, long long *launches);
cudaError_t launch_wait_probe(photon_ctx *ctx, unsigned long long limit_ns, cudaStream_t st, long long *launches);

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
