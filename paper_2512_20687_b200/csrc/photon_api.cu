// C boundary: context management, argument validation, launch sequencing.
#include <chrono>
#include <algorithm>
#include <cstdio>
#include <new>

#include "common.cuh"

namespace {

constexpr int kDefaultMaxSplits = 32;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool kv_ok(const photon_ctx *ctx, const photon_kv *c, bool allow_shared) {
    if (!c || !c->k || !c->v || !c->len) return false;
    if (!aligned16(c->k) || !aligned16(c->v)) return false;
    if (c->n_units < 0 || c->cap <= 0 || c->max_len < 0 || c->max_len > c->cap) return false;
    if (c->k_shared) {
        if (!allow_shared) return false;
        if (!c->v_shared || !c->shared_len || !c->shared_id) return false;
        if (!aligned16(c->k_shared) || !aligned16(c->v_shared)) return false;
        if (c->n_shared <= 0 || c->cap_shared <= 0 || c->max_shared_len < 0 ||
            c->max_shared_len > c->cap_shared)
            return false;
    }
    if (c->page_table) {
        if (c->page_rows <= 0 || c->page_rows % 64 != 0 || c->pages_per_unit <= 0 || c->n_pages <= 0) return false;
        if ((int64_t)c->page_rows * c->pages_per_unit != c->cap) return false;
    }
    (void)ctx;
    return true;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }


// k_new, v_new: the step's append folded into the attention over the units' own keys (see AttnParams), or NULL.
photon_status attention_common(photon_ctx *ctx, const photon_kv *cache, const photon_bf16 *q,
                               const int32_t *slot, int n_q, photon_bf16 *out, float *lse,
                               float scale, bool chunk, cudaStream_t st, const photon_bf16 *k_new = nullptr,
                               const photon_bf16 *v_new = nullptr) {
    if (!ctx) return PHOTON_ERR_INVALID_ARG;
    if (!kv_ok(ctx, cache, !chunk) || (chunk && cache->page_table)) return PHOTON_ERR_INVALID_ARG;
    if (n_q < 0 || (n_q > 0 && (!q || !out))) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out)) return PHOTON_ERR_INVALID_ARG;
    if (!(scale == scale)) return PHOTON_ERR_INVALID_ARG;
    if (n_q == 0) return PHOTON_OK;
    const photon_config &c = ctx->cfg;
    // TMA row coordinates are 32-bit
    const uint64_t pool_rows = cache->page_table ? (uint64_t)cache->n_pages * c.Hkv * cache->page_rows
                                                 : (uint64_t)cache->n_units * c.Hkv * cache->cap;
    if (pool_rows >= (1ull << 31)) return PHOTON_ERR_UNSUPPORTED;
    if (cache->k_shared && (uint64_t)cache->n_shared * c.Hkv * cache->cap_shared >= (1ull << 31))
        return PHOTON_ERR_UNSUPPORTED;
    AttnParams p{};
    p.q = reinterpret_cast<const bf16 *>(q);
    p.out = reinterpret_cast<bf16 *>(out);
    p.lse = lse;
    p.k = reinterpret_cast<const bf16 *>(cache->k);
    p.v = reinterpret_cast<const bf16 *>(cache->v);
    p.len = cache->len;
    p.n_units = cache->n_units;
    p.cap = cache->cap;
    p.slot = slot;
    p.page_table = cache->page_table;
    p.page_rows = cache->page_rows; p.pages_per_unit = cache->pages_per_unit; p.n_pages = cache->n_pages;
    p.n_q = n_q;
    p.Hq = c.Hq; p.Hkv = c.Hkv; p.dh = c.dh;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.partials = ctx->partials;
    p.tickets = ctx->tickets;
    p.status = ctx->status;

    p.cta_partials = ctx->cta_partials;
    if (k_new) {
        p.k_new = reinterpret_cast<const bf16 *>(k_new);
        p.v_new = reinterpret_cast<const bf16 *>(v_new);
        p.k_w = reinterpret_cast<bf16 *>(cache->k);
        p.v_w = reinterpret_cast<bf16 *>(cache->v);
        p.len_w = cache->len;
        p.readers = ctx->readers;
    }
    p.max_len = cache->max_len ? cache->max_len : cache->cap;
    p.splits_sh = 0;
    if (!chunk) {
        if ((size_t)n_q * c.Hkv > ctx->n_tickets) return PHOTON_ERR_WORKSPACE;
        if (cache->k_shared) {
            p.ks = reinterpret_cast<const bf16 *>(cache->k_shared);
            p.vs = reinterpret_cast<const bf16 *>(cache->v_shared);
            p.sh_len = cache->shared_len; p.sh_id = cache->shared_id;
            p.n_shared = cache->n_shared; p.cap_sh = cache->cap_shared;
            const int ms = cache->max_shared_len ? cache->max_shared_len : cache->cap_shared;
            if (size_t(n_q) * c.Hq * (c.dh + 2) > ctx->partial_floats) return PHOTON_ERR_WORKSPACE;
            const int G = c.Hq / c.Hkv;
            const int groups = ceil_div(n_q, shared_prefix_units_per_cta(G));     // tiles of 128 query rows
            // key ranges per row tile = cluster size: a power of two up to 8, about one wave of CTAs in all
            const int want = std::max(1, ctx->sm_count / std::max(1, groups * c.Hkv));
            const int cap = std::min(std::min(want, std::max(1, ms / 128)), std::min(8, ctx->max_splits));
            p.splits_sh = 1;
            while (p.splits_sh * 2 <= cap) p.splits_sh *= 2;
        }
    }
    const cudaError_t e = chunk ? launch_chunk_attention(ctx, p, st, &ctx->launches)
                                : launch_attention(ctx, p, st, &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

}  // namespace

extern "C" {

photon_status photon_create(photon_ctx **out, const photon_config *cfg) {
    if (!out) return PHOTON_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = *cfg;
    if (c.Hq <= 0 || c.Hkv <= 0 || c.dh <= 0 || c.D <= 0 || c.P <= 0 || c.C <= 0 ||
        c.max_queries <= 0 || c.max_splits < 0)
        return PHOTON_ERR_INVALID_ARG;
    if (c.Hq % c.Hkv != 0) return PHOTON_ERR_INVALID_ARG;
    if (c.dh != 64 && c.dh != 128) return PHOTON_ERR_UNSUPPORTED;
    if (c.Hq / c.Hkv > 16 || c.D % 64 != 0 || c.P + c.C > 64) return PHOTON_ERR_UNSUPPORTED;

    photon_ctx *ctx = new (std::nothrow) photon_ctx();
    if (!ctx) return PHOTON_ERR_CUDA;
    ctx->cfg = c;
    ctx->max_splits = c.max_splits ? c.max_splits : kDefaultMaxSplits;
    ctx->launches = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&ctx->device) != cudaSuccess ||
        cudaGetDeviceProperties(&prop, ctx->device) != cudaSuccess) {
        delete ctx;
        return PHOTON_ERR_CUDA;
    }
    if (prop.major != 10) {              // built for sm_100a only
        delete ctx;
        return PHOTON_ERR_UNSUPPORTED;
    }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->partial_floats = size_t(c.max_queries) * c.Hq * (c.dh + 2);      // one shared-prefix partial per query head
    ctx->n_tickets = size_t(c.max_queries) * c.Hkv;
    ctx->max_ctas = ctx->sm_count * coarse_attn_ctas_per_sm();
    ctx->attn_ctas = 0;
    ctx->host_pause_ns = 1500;
    ctx->host_poll_us = 2000;
    if (cudaMalloc(&ctx->partials, ctx->partial_floats * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ctx->cta_partials, size_t(2) * ctx->max_ctas * 16 * (c.dh + 2) * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ctx->tickets, ctx->n_tickets * sizeof(int32_t)) != cudaSuccess ||
        cudaMalloc(&ctx->status, 64 * sizeof(int32_t)) != cudaSuccess ||     // the word, and the counters 128 B on
        cudaMemset(ctx->tickets, 0, ctx->n_tickets * sizeof(int32_t)) != cudaSuccess ||
        cudaMemset(ctx->status, 0, 64 * sizeof(int32_t)) != cudaSuccess) {
        cudaFree(ctx->partials); cudaFree(ctx->cta_partials); cudaFree(ctx->tickets); cudaFree(ctx->status);
        cudaGetLastError();
        delete ctx;
        return PHOTON_ERR_CUDA;
    }
    ctx->work = ctx->status + 32;
    ctx->readers = ctx->status + 40;
    int lo = 0, hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess ||
        cudaStreamCreateWithPriority(&ctx->side, cudaStreamNonBlocking, lo) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaStreamCreateWithFlags(&ctx->copy, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_mid, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_copy, cudaEventDisableTiming) != cudaSuccess) {
        photon_destroy(ctx);
        cudaGetLastError();
        return PHOTON_ERR_CUDA;
    }
    *out = ctx;
    return PHOTON_OK;
}

photon_status photon_destroy(photon_ctx *ctx) {
    if (!ctx) return PHOTON_ERR_INVALID_ARG;
    cudaFree(ctx->partials);
    cudaFree(ctx->cta_partials);
    cudaFree(ctx->tickets);
    cudaFree(ctx->status);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    if (ctx->ev_mid) cudaEventDestroy(ctx->ev_mid);
    if (ctx->ev_copy) cudaEventDestroy(ctx->ev_copy);
    if (ctx->copy) cudaStreamDestroy(ctx->copy);
    delete ctx;
    return PHOTON_OK;
}

photon_status photon_kv_append(photon_ctx *ctx, photon_kv *cache, const photon_bf16 *k_new,
                               const photon_bf16 *v_new, const int32_t *unit_ids, int32_t n,
                               int32_t n_rows, photon_stream stream) {
    if (!ctx || !kv_ok(ctx, cache, true)) return PHOTON_ERR_INVALID_ARG;
    if (n < 0 || n_rows <= 0 || n_rows > cache->cap) return PHOTON_ERR_INVALID_ARG;
    if (n > 0 && (!k_new || !v_new)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new)) return PHOTON_ERR_INVALID_ARG;
    if (!unit_ids && n > cache->n_units) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    const cudaError_t e = launch_kv_append(
        reinterpret_cast<bf16 *>(cache->k), reinterpret_cast<bf16 *>(cache->v), cache->len,
        cache->n_units, c.Hkv, cache->cap, c.dh, reinterpret_cast<const bf16 *>(k_new),
        reinterpret_cast<const bf16 *>(v_new), unit_ids, n, n_rows,
        Paging{cache->page_table, cache->page_rows, cache->pages_per_unit, cache->n_pages}, ctx->status,
        static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_coarse_attn(photon_ctx *ctx, const photon_kv *cache, const photon_bf16 *q,
                                 photon_bf16 *out, float *lse, float scale, photon_stream stream) {
    if (!cache) return PHOTON_ERR_INVALID_ARG;
    return attention_common(ctx, cache, q, nullptr, cache->n_units, out, lse, scale, false,
                            static_cast<cudaStream_t>(stream));
}

photon_status photon_flat_attn(photon_ctx *ctx, const photon_kv *cache, const photon_bf16 *q,
                               photon_bf16 *out, float *lse, float scale, photon_stream stream) {
    if (!cache) return PHOTON_ERR_INVALID_ARG;
    return attention_common(ctx, cache, q, nullptr, cache->n_units, out, lse, scale, false,
                            static_cast<cudaStream_t>(stream));
}

photon_status photon_chunk_attn(photon_ctx *ctx, const photon_kv *chunks, const photon_bf16 *q,
                                const int32_t *slot, photon_bf16 *out, int32_t Nc, float scale,
                                photon_stream stream) {
    if (!ctx || !chunks) return PHOTON_ERR_INVALID_ARG;
    if (chunks->cap > ctx->cfg.P + ctx->cfg.C) return PHOTON_ERR_INVALID_ARG;
    if (!slot && Nc > chunks->n_units) return PHOTON_ERR_INVALID_ARG;
    return attention_common(ctx, chunks, q, slot, Nc, out, nullptr, scale, true,
                            static_cast<cudaStream_t>(stream));
}

photon_status photon_chunk_causal_attn(photon_ctx *ctx, const photon_kv *chunks, const photon_bf16 *q,
                                       const int32_t *slot, photon_bf16 *out, int32_t Nc, int32_t row0,
                                       int32_t rows, float scale, photon_stream stream) {
    if (!ctx || !chunks) return PHOTON_ERR_INVALID_ARG;
    if (!kv_ok(ctx, chunks, false) || chunks->page_table) return PHOTON_ERR_INVALID_ARG;
    if (chunks->cap > ctx->cfg.P + ctx->cfg.C || chunks->cap > 64) return PHOTON_ERR_INVALID_ARG;
    if (Nc < 0 || row0 < 0 || rows < 1 || row0 + rows > chunks->cap) return PHOTON_ERR_INVALID_ARG;
    if (!slot && Nc > chunks->n_units) return PHOTON_ERR_INVALID_ARG;
    if (Nc > 0 && (!q || !out)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !(scale == scale)) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    CausalParams p{};
    p.q = reinterpret_cast<const bf16 *>(q);
    p.out = reinterpret_cast<bf16 *>(out);
    p.k = reinterpret_cast<const bf16 *>(chunks->k);
    p.v = reinterpret_cast<const bf16 *>(chunks->v);
    p.len = chunks->len;
    p.slot = slot;
    p.n_units = chunks->n_units; p.cap = chunks->cap;
    p.n = Nc; p.R = rows; p.row0 = row0;
    p.Hq = c.Hq; p.Hkv = c.Hkv; p.dh = c.dh;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = ctx->status;
    const cudaError_t e = launch_chunk_causal_attention(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_converter(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *w,
                               int32_t w_layout, const photon_bf16 *bias, photon_bf16 *U, int32_t B,
                               photon_stream stream) {
    if (!ctx || B < 0) return PHOTON_ERR_INVALID_ARG;
    if (B > 0 && (!x || !w || !U)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(U) || !aligned16(bias))
        return PHOTON_ERR_INVALID_ARG;
    if (w_layout != PHOTON_W_IN_MAJOR && w_layout != PHOTON_W_OUT_MAJOR)
        return PHOTON_ERR_INVALID_ARG;
    ConvParams p{};
    p.x = reinterpret_cast<const bf16 *>(x);
    p.w = reinterpret_cast<const bf16 *>(w);
    p.bias = reinterpret_cast<const bf16 *>(bias);
    p.U = reinterpret_cast<bf16 *>(U);
    p.B = B; p.D = ctx->cfg.D; p.N = ctx->cfg.P * ctx->cfg.D;
    p.w_out_major = (w_layout == PHOTON_W_OUT_MAJOR);
    p.status = ctx->status;
    const cudaError_t e = linear_wants_large_tiles(ctx, p)      // batches of more than a thousand latents
                              ? launch_linear_large(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches)
                              : launch_converter(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_rmsnorm(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *gamma, float eps,
                             photon_bf16 *out, int32_t rows, int32_t cols, photon_stream stream) {
    if (!ctx || rows < 0 || cols <= 0 || cols % 8 != 0) return PHOTON_ERR_INVALID_ARG;
    if (rows > 0 && (!x || !out)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(out) || !(eps >= 0.f)) return PHOTON_ERR_INVALID_ARG;
    const cudaError_t e = launch_rmsnorm(reinterpret_cast<const bf16 *>(x), reinterpret_cast<const bf16 *>(gamma), eps,
                                         reinterpret_cast<bf16 *>(out), rows, cols,
                                         static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_linear(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *w, int32_t w_layout,
                            const photon_bf16 *bias, const photon_bf16 *residual, photon_bf16 *y, int32_t B,
                            int32_t K, int32_t N, photon_stream stream) {
    if (!ctx || B < 0 || K <= 0 || N <= 0 || K % 64 != 0 || N % 64 != 0) return PHOTON_ERR_INVALID_ARG;
    if (B > 0 && (!x || !w || !y)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(bias) || !aligned16(residual))
        return PHOTON_ERR_INVALID_ARG;
    if (w_layout != PHOTON_W_IN_MAJOR && w_layout != PHOTON_W_OUT_MAJOR) return PHOTON_ERR_INVALID_ARG;
    ConvParams p{};
    p.x = reinterpret_cast<const bf16 *>(x);
    p.w = reinterpret_cast<const bf16 *>(w);
    p.bias = reinterpret_cast<const bf16 *>(bias);
    p.residual = reinterpret_cast<const bf16 *>(residual);
    p.U = reinterpret_cast<bf16 *>(y);
    p.B = B; p.D = K; p.N = N;
    p.w_out_major = (w_layout == PHOTON_W_OUT_MAJOR);
    p.status = ctx->status;
    // thousands of rows: the persistent kernel with two accumulators in TMEM; else the converter's kernel
    const cudaError_t e = linear_wants_large_tiles(ctx, p)
                              ? launch_linear_large(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches)
                              : launch_linear(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_rope_split(photon_ctx *ctx, const photon_bf16 *qkv, const int32_t *pos, int32_t n,
                                float theta, photon_bf16 *q, photon_bf16 *k, photon_bf16 *v,
                                photon_stream stream) {
    if (!ctx || n < 0 || !(theta > 1.f)) return PHOTON_ERR_INVALID_ARG;
    if (n > 0 && (!qkv || !pos || !q || !k || !v)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(q) || !aligned16(k) || !aligned16(v)) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    const cudaError_t e = launch_rope_split(reinterpret_cast<const bf16 *>(qkv), pos, 1, n, c.Hq, c.Hkv, c.dh, theta,
                                            reinterpret_cast<bf16 *>(q), reinterpret_cast<bf16 *>(k),
                                            reinterpret_cast<bf16 *>(v), static_cast<cudaStream_t>(stream),
                                            &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_swiglu(photon_ctx *ctx, const photon_bf16 *gu, photon_bf16 *out, int32_t n, int32_t F,
                            photon_stream stream) {
    if (!ctx || n < 0 || F <= 0 || F % 8 != 0) return PHOTON_ERR_INVALID_ARG;
    if (n > 0 && (!gu || !out)) return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(gu) || !aligned16(out)) return PHOTON_ERR_INVALID_ARG;
    const cudaError_t e = launch_swiglu(reinterpret_cast<const bf16 *>(gu), reinterpret_cast<bf16 *>(out), n, F,
                                        static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

namespace {
// gate/up projection and activation: act [rows, F] = silu(n Wg) * (n Wu).  One fused launch (gu is then not written)
// of the large-tile kernel with thousands of rows, of the slab kernel where 64-feature slabs occupy most of the GPU;
// else the projection followed by photon_swiglu.
photon_status gate_up(photon_ctx *ctx, const photon_layer *L, const photon_layer_scratch *sc, int rows,
                      photon_stream stream) {
    const photon_config &c = ctx->cfg;
    ConvParams p{};
    p.x = reinterpret_cast<const bf16 *>(sc->n);
    p.w = reinterpret_cast<const bf16 *>(L->wgu);
    p.U = reinterpret_cast<bf16 *>(sc->act);
    p.B = rows; p.D = c.D; p.N = 2 * L->F;
    p.w_out_major = (L->w_layout == PHOTON_W_OUT_MAJOR);
    p.status = ctx->status;
    if (L->F % 128 == 0 && linear_wants_large_tiles(ctx, p)) {
        const cudaError_t e = launch_gate_up_large(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches);
        return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
    }
    if (gate_up_fits_small_tiles(ctx, p)) {                                // one launch, gu is not written
        const cudaError_t e = launch_gate_up(ctx, p, static_cast<cudaStream_t>(stream), &ctx->launches);
        return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
    }
    photon_status s = photon_linear(ctx, sc->n, L->wgu, L->w_layout, nullptr, nullptr, sc->gu, rows, c.D, 2 * L->F, stream);
    if (s == PHOTON_OK) s = photon_swiglu(ctx, sc->gu, sc->act, rows, L->F, stream);
    return s;
}

// STEP of one layer for the newest position of every unit of `cache`; local: the cache is a set of chunk
// buffers read by the chunk attention, else a coarse stream read by the coarse attention.
photon_status layer_step(photon_ctx *ctx, const photon_layer *L, const photon_layer_scratch *sc,
                         const photon_bf16 *x, photon_kv *cache, photon_bf16 *y, float scale, bool local,
                         photon_stream stream) {
    if (!ctx || !L || !sc || !cache || !x || !y) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    // everything is validated before the first launch, so that a bad argument leaves no partial step behind
    if (!kv_ok(ctx, cache, false) || c.Hq * c.dh != c.D || L->F <= 0 || L->F % 64 != 0) return PHOTON_ERR_INVALID_ARG;
    if (!L->g1 || !L->wqkv || !L->wo || !L->g2 || !L->wgu || !L->wdown || !(L->eps >= 0.f) || !(L->theta > 1.f))
        return PHOTON_ERR_INVALID_ARG;
    if (L->w_layout != PHOTON_W_IN_MAJOR && L->w_layout != PHOTON_W_OUT_MAJOR) return PHOTON_ERR_INVALID_ARG;
    const void *ptrs[] = {L->g1, L->wqkv, L->wo, L->g2, L->wgu, L->wdown, sc->n, sc->qkv, sc->q, sc->k_new,
                          sc->v_new, sc->att, sc->h, sc->gu, sc->act, x, y};
    for (const void *q : ptrs)
        if (!q || !aligned16(q)) return PHOTON_ERR_INVALID_ARG;
    const int B = cache->n_units, D = c.D, QKV = (c.Hq + 2 * c.Hkv) * c.dh;
    if (!local && (size_t)B * c.Hkv > ctx->n_tickets) return PHOTON_ERR_WORKSPACE;
    if (local && (cache->cap > c.P + c.C || cache->page_table)) return PHOTON_ERR_INVALID_ARG;
    photon_status s = photon_rmsnorm(ctx, x, L->g1, L->eps, sc->n, B, D, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->n, L->wqkv, L->w_layout, nullptr, nullptr, sc->qkv, B, D, QKV, stream);
    if (s == PHOTON_OK) {
        // split, rotation by the unit's length and the append in one kernel: k and v go straight into the cache rows
        const cudaError_t e = launch_rope_split_append(
            reinterpret_cast<const bf16 *>(sc->qkv), B, c.Hq, c.Hkv, c.dh, L->theta, reinterpret_cast<bf16 *>(sc->q),
            reinterpret_cast<bf16 *>(cache->k), reinterpret_cast<bf16 *>(cache->v), cache->len, cache->cap,
            Paging{cache->page_table, cache->page_rows, cache->pages_per_unit, cache->n_pages}, ctx->status,
            static_cast<cudaStream_t>(stream), &ctx->launches);
        if (e != cudaSuccess) s = PHOTON_ERR_CUDA;
    }
    if (s == PHOTON_OK)
        s = local ? photon_chunk_attn(ctx, cache, sc->q, nullptr, sc->att, B, scale, stream)
                  : photon_coarse_attn(ctx, cache, sc->q, sc->att, nullptr, scale, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->att, L->wo, L->w_layout, nullptr, x, sc->h, B, D, D, stream);
    if (s == PHOTON_OK) s = photon_rmsnorm(ctx, sc->h, L->g2, L->eps, sc->n, B, D, stream);
    if (s == PHOTON_OK) s = gate_up(ctx, L, sc, B, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->act, L->wdown, L->w_layout, nullptr, sc->h, y, B, L->F, D, stream);
    return s;
}
}  // namespace

photon_status photon_encoder_step(photon_ctx *ctx, const photon_layer *layer, const photon_layer_scratch *scratch,
                                  const photon_bf16 *x, photon_kv *cache, photon_bf16 *y, float scale,
                                  photon_stream stream) {
    return layer_step(ctx, layer, scratch, x, cache, y, scale, false, stream);
}

photon_status photon_decoder_prefill(photon_ctx *ctx, const photon_layer *L, const photon_layer_scratch *sc,
                                     const photon_bf16 *U, photon_kv *chunks, const int32_t *unit_ids, int32_t n,
                                     photon_bf16 *y, float scale, photon_stream stream) {
    if (!ctx || !L || !sc || !chunks || n < 0) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    if (!kv_ok(ctx, chunks, false) || chunks->page_table || c.Hq * c.dh != c.D || L->F <= 0 || L->F % 64 != 0)
        return PHOTON_ERR_INVALID_ARG;
    if (chunks->cap > c.P + c.C || chunks->cap > 64 || c.P > chunks->cap) return PHOTON_ERR_INVALID_ARG;
    if (!unit_ids && n > chunks->n_units) return PHOTON_ERR_INVALID_ARG;
    if (!L->g1 || !L->wqkv || !L->wo || !L->g2 || !L->wgu || !L->wdown || !(L->eps >= 0.f) || !(L->theta > 1.f))
        return PHOTON_ERR_INVALID_ARG;
    if (L->w_layout != PHOTON_W_IN_MAJOR && L->w_layout != PHOTON_W_OUT_MAJOR) return PHOTON_ERR_INVALID_ARG;
    const void *ptrs[] = {L->g1, L->wqkv, L->wo, L->g2, L->wgu, L->wdown, sc->n, sc->qkv, sc->q, sc->k_new,
                          sc->v_new, sc->att, sc->h, sc->gu, sc->act, U, y};
    for (const void *q : ptrs)
        if (!q || !aligned16(q)) return PHOTON_ERR_INVALID_ARG;
    if (n == 0) return PHOTON_OK;
    const int P = c.P, T = n * P, D = c.D, QKV = (c.Hq + 2 * c.Hkv) * c.dh;      // T rows: the P prefix vectors of n chunks
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    photon_status s = photon_rmsnorm(ctx, U, L->g1, L->eps, sc->n, T, D, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->n, L->wqkv, L->w_layout, nullptr, nullptr, sc->qkv, T, D, QKV, stream);
    if (s == PHOTON_OK &&
        launch_rope_split(reinterpret_cast<const bf16 *>(sc->qkv), nullptr, P, T, c.Hq, c.Hkv, c.dh, L->theta,
                          reinterpret_cast<bf16 *>(sc->q), reinterpret_cast<bf16 *>(sc->k_new),
                          reinterpret_cast<bf16 *>(sc->v_new), st, &ctx->launches) != cudaSuccess)
        s = PHOTON_ERR_CUDA;
    if (s == PHOTON_OK) s = photon_kv_append(ctx, chunks, sc->k_new, sc->v_new, unit_ids, n, P, stream);
    if (s == PHOTON_OK) s = photon_chunk_causal_attn(ctx, chunks, sc->q, unit_ids, sc->att, n, 0, P, scale, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->att, L->wo, L->w_layout, nullptr, U, sc->h, T, D, D, stream);
    if (s == PHOTON_OK) s = photon_rmsnorm(ctx, sc->h, L->g2, L->eps, sc->n, T, D, stream);
    if (s == PHOTON_OK) s = gate_up(ctx, L, sc, T, stream);
    if (s == PHOTON_OK) s = photon_linear(ctx, sc->act, L->wdown, L->w_layout, nullptr, sc->h, y, T, L->F, D, stream);
    return s;
}

photon_status photon_decoder_step(photon_ctx *ctx, const photon_layer *layer, const photon_layer_scratch *scratch,
                                  const photon_bf16 *x, photon_kv *chunks, photon_bf16 *y, float scale,
                                  photon_stream stream) {
    return layer_step(ctx, layer, scratch, x, chunks, y, scale, true, stream);
}

namespace {
// Host buffers of a step: [0, in_split) of the input is what the coarse part reads, the rest what only the
// chunk attention reads; [0, out_split) of the output is what the coarse part writes, the rest the chunk attention's.
struct HostPlan {
    const char *host_in;
    char *dev_in;
    size_t in_bytes, in_split;
    const char *dev_out;
    char *host_out;
    size_t out_bytes, out_split;
};

// The address under which kernels can reach page-locked, mapped host memory; nullptr for any other memory.
// Asked every time: an address can come back from the allocator as another kind of memory.
char *device_alias(const void *host) {
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, host) == cudaSuccess && at.type == cudaMemoryTypeHost)
        return static_cast<char *>(at.devicePointer);
    cudaGetLastError();
    return nullptr;
}

bool inside(const void *p, size_t n, const char *base, size_t from, size_t to) {
    const char *c = static_cast<const char *>(p);
    return c >= base + from && c + n <= base + to;
}

bool copy_in(const HostPlan *hp, size_t from, size_t to, cudaStream_t st) {
    return to <= from || cudaMemcpyAsync(hp->dev_in + from, hp->host_in + from, to - from, cudaMemcpyHostToDevice, st) == cudaSuccess;
}
bool copy_out(const HostPlan *hp, size_t from, size_t to, cudaStream_t st) {
    return to <= from || cudaMemcpyAsync(hp->host_out + from, hp->dev_out + from, to - from, cudaMemcpyDeviceToHost, st) == cudaSuccess;
}

photon_status step_impl(photon_ctx *ctx, const photon_step_args *a, photon_stream stream, const HostPlan *hp) {
    if (!ctx || !a || !a->coarse) return PHOTON_ERR_INVALID_ARG;
    const photon_config &c = ctx->cfg;
    const bool chain = (a->x == nullptr);
    // validate everything before the first launch so that a bad argument leaves no partial step behind
    if (!kv_ok(ctx, a->coarse, true) || !a->k_new || !a->v_new || !a->q_coarse || !a->out_coarse)
        return PHOTON_ERR_INVALID_ARG;
    if (!aligned16(a->k_new) || !aligned16(a->v_new) || !aligned16(a->q_coarse) ||
        !aligned16(a->out_coarse))
        return PHOTON_ERR_INVALID_ARG;
    if (!a->w || !a->U || a->B < 0 || !aligned16(a->w) || !aligned16(a->U) || !aligned16(a->x) ||
        !aligned16(a->bias))
        return PHOTON_ERR_INVALID_ARG;
    if (a->w_layout != PHOTON_W_IN_MAJOR && a->w_layout != PHOTON_W_OUT_MAJOR)
        return PHOTON_ERR_INVALID_ARG;
    if (chain && (c.Hq * c.dh != c.D || a->B != a->coarse->n_units)) return PHOTON_ERR_INVALID_ARG;
    if (a->Nc < 0) return PHOTON_ERR_INVALID_ARG;
    if (a->Nc > 0) {
        if (!kv_ok(ctx, a->chunks, false) || !a->q_chunk || !a->out_chunk ||
            !aligned16(a->q_chunk) || !aligned16(a->out_chunk))
            return PHOTON_ERR_INVALID_ARG;
        if (a->chunks->cap > c.P + c.C || (!a->slot && a->Nc > a->chunks->n_units))
            return PHOTON_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The chunk attention shares no data with the other parts (the decoders' projections, which are not
    // built, sit between the converter's output and the chunk caches): it runs beside them on a
    // low-priority stream that forks from `stream` here and joins it again before the call returns, so
    // for the caller the whole step is still ordered on `stream`.  Large chunk workloads stay in line:
    // two kernels that are both bound by HBM gain nothing from running side by side.
    const bool beside = a->Nc > 0 &&
                        (size_t)a->Nc * c.Hkv * a->chunks->cap * c.dh * 4 <= (size_t(32) << 20);
    photon_status s = PHOTON_OK;
    // With host buffers and a declared split the two halves of either buffer travel apart.  Where both host buffers are
    // mapped into the device and the chunk attention's arrays lie wholly in its halves of the staging areas, that
    // kernel reads its queries from and writes its results to the host buffers themselves: no copy, and no hand-over
    // between the copy engines and the SMs, for those bytes (direct).  Otherwise, with the chunk attention on its own
    // stream, its inputs follow the coarse part's over the bus while the append and the coarse attention already run
    // and its results leave when it ends.  The coarse results leave beside the converter in both cases (apart).
    const bool split = hp && a->Nc > 0 && (hp->in_split < hp->in_bytes || hp->out_split < hp->out_bytes);
    const bool apart = split && beside;
    const photon_bf16 *q_chunk = a->q_chunk;
    const int32_t *slot = a->slot;
    photon_bf16 *out_chunk = a->out_chunk;
    bool direct = false;
    // Beside the coarse part only small chunk workloads go direct: a kernel that waits for the bus keeps its CTAs
    // resident for as long as the transfer takes, and they stand in the way of the coarse part's kernels (measured with
    // 2 MB each way on the shared-prefix workload: 155-269 us per step, unstable, against 154 us with copies; with
    // 0.5 MB on the default workload: 65 against 67-78 us).  In line nothing runs beside it.
    const size_t qb_all = (size_t)a->Nc * c.Hq * c.dh * sizeof(photon_bf16);
    if (split && (!beside || qb_all <= (size_t(1) << 20))) {
        const size_t qb = qb_all, sb = (size_t)a->Nc * sizeof(int32_t);
        const bool slot_in = slot && inside(slot, sb, hp->dev_in, hp->in_split, hp->in_bytes);
        const bool slot_off = !slot || (const char *)slot + sb <= hp->dev_in || (const char *)slot >= hp->dev_in + hp->in_bytes;
        if (inside(q_chunk, qb, hp->dev_in, hp->in_split, hp->in_bytes) &&
            inside(out_chunk, qb, hp->dev_out, hp->out_split, hp->out_bytes) && (slot_in || slot_off)) {
            char *in_alias = device_alias(hp->host_in), *out_alias = device_alias(hp->host_out);
            if (in_alias && out_alias) {
                direct = true;
                q_chunk = reinterpret_cast<const photon_bf16 *>(in_alias + ((const char *)q_chunk - hp->dev_in));
                out_chunk = reinterpret_cast<photon_bf16 *>(out_alias + ((const char *)out_chunk - hp->dev_out));
                if (slot_in) slot = reinterpret_cast<const int32_t *>(in_alias + ((const char *)slot - hp->dev_in));
            }
        }
    }
    // A chunk attention that reads its queries (and slots) from the host buffer itself and whose lengths lie outside the
    // staging area needs nothing of this call's copy: its stream forks before the copy is enqueued, not after it.
    bool forked = false;
    if (beside && direct) {
        const char *cl = reinterpret_cast<const char *>(a->chunks->len);
        const bool len_off = cl + (size_t)a->chunks->n_units * sizeof(int32_t) <= hp->dev_in || cl >= hp->dev_in + hp->in_bytes;
        if (len_off) {
            if (cudaEventRecord(ctx->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess)
                return PHOTON_ERR_CUDA;
            forked = true;
        }
    }
    if (hp) {
        if (!copy_in(hp, 0, apart || direct ? hp->in_split : hp->in_bytes, st)) return PHOTON_ERR_CUDA;
        if (hp->in_bytes && ctx->host_pause_ns > 0) {
            // Measured on one host: launches enqueued within a microsecond of the copy make the whole step finish about
            // 5 us later than launches that follow 1.5 us behind it (a stream query in between does not help, a pause
            // does).  The length of the pause is the context's (photon_set_host_step_tuning; 0 switches it off).
            const auto g0 = std::chrono::steady_clock::now();
            while (std::chrono::steady_clock::now() - g0 < std::chrono::nanoseconds(ctx->host_pause_ns)) {}
        }
    }
    if (beside) {
        if (!forked && (cudaEventRecord(ctx->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess))
            return PHOTON_ERR_CUDA;
        if (apart && !direct && !copy_in(hp, hp->in_split, hp->in_bytes, ctx->side)) s = PHOTON_ERR_CUDA;
        if (s == PHOTON_OK)
            s = photon_chunk_attn(ctx, a->chunks, q_chunk, slot, out_chunk, a->Nc, a->scale_chunk, ctx->side);
        if (s == PHOTON_OK && apart && !direct && !copy_out(hp, hp->out_split, hp->out_bytes, ctx->side)) s = PHOTON_ERR_CUDA;
        // every way out from here on joins the side stream again, failed calls included
        if (cudaEventRecord(ctx->ev_join, ctx->side) != cudaSuccess) s = PHOTON_ERR_CUDA;
        if (s != PHOTON_OK) { cudaStreamWaitEvent(st, ctx->ev_join, 0); return s; }
    }
    // The append is one row per unit, in place: for a contiguous cache of a batch whose lengths fit the attention
    // kernel's shared memory it is folded into that kernel (the warp that reaches a unit's last tile installs the
    // new row in the tile and in the cache; the lengths grow once every CTA has read them), which takes a launch
    // and the wait between two launches out of the step.  Otherwise the append is its own kernel.
    // (Not where short own caches ride along in the shared-prefix kernel: that path has no kernel of own keys to fold into.)
    const bool fold = !a->coarse->page_table && a->coarse->n_units <= coarse_attn_fold_limit() &&
                      !own_keys_ride_with_prefix(a->coarse);
    if (!fold) s = photon_kv_append(ctx, a->coarse, a->k_new, a->v_new, nullptr, a->coarse->n_units, 1, stream);
    if (s == PHOTON_OK && a->ev_attn_begin && cudaEventRecord(static_cast<cudaEvent_t>(a->ev_attn_begin), st) != cudaSuccess)
        s = PHOTON_ERR_CUDA;
    if (s == PHOTON_OK)
        s = fold ? attention_common(ctx, a->coarse, a->q_coarse, nullptr, a->coarse->n_units, a->out_coarse, a->lse_coarse,
                                    a->scale_coarse, false, st, a->k_new, a->v_new)
                 : photon_coarse_attn(ctx, a->coarse, a->q_coarse, a->out_coarse, a->lse_coarse, a->scale_coarse, stream);
    if (s == PHOTON_OK && a->ev_attn_end && cudaEventRecord(static_cast<cudaEvent_t>(a->ev_attn_end), st) != cudaSuccess)
        s = PHOTON_ERR_CUDA;
    // What the coarse attention wrote leaves beside the converter.  Where the converter's own output lies in the
    // coarse part of the staging area, it and whatever follows it there leave after the converter.
    size_t early_end = hp ? hp->out_split : 0;
    if (hp && inside(a->U, (size_t)a->B * c.P * c.D * sizeof(photon_bf16), hp->dev_out, 0, hp->out_split))
        early_end = (size_t)(reinterpret_cast<const char *>(a->U) - hp->dev_out);
    bool copying = false;
    if (s == PHOTON_OK && (apart || direct) && early_end > 0) {
        if (cudaEventRecord(ctx->ev_mid, st) != cudaSuccess || cudaStreamWaitEvent(ctx->copy, ctx->ev_mid, 0) != cudaSuccess)
            s = PHOTON_ERR_CUDA;
        else {
            copying = true;
            if (!copy_out(hp, 0, early_end, ctx->copy)) s = PHOTON_ERR_CUDA;
            if (cudaEventRecord(ctx->ev_copy, ctx->copy) != cudaSuccess) s = PHOTON_ERR_CUDA;
        }
    }
    if (s == PHOTON_OK)
        s = photon_converter(ctx, chain ? a->out_coarse : a->x, a->w, a->w_layout, a->bias, a->U, a->B, stream);
    if (beside) {
        if (cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess && s == PHOTON_OK) s = PHOTON_ERR_CUDA;
    } else if (s == PHOTON_OK && a->Nc > 0) {
        s = photon_chunk_attn(ctx, a->chunks, q_chunk, slot, out_chunk, a->Nc, a->scale_chunk, stream);
    }
    if (copying && cudaStreamWaitEvent(st, ctx->ev_copy, 0) != cudaSuccess && s == PHOTON_OK) s = PHOTON_ERR_CUDA;
    if (s == PHOTON_OK && hp && !copy_out(hp, copying ? early_end : 0, apart || direct ? hp->out_split : hp->out_bytes, st))
        s = PHOTON_ERR_CUDA;
    return s;
}
}  // namespace

photon_status photon_decode_step(photon_ctx *ctx, const photon_step_args *a, photon_stream stream) {
    return step_impl(ctx, a, stream, nullptr);
}

photon_status photon_decode_step_host(photon_ctx *ctx, const photon_step_args *args, const void *host_in,
                                      void *dev_in, size_t in_bytes, size_t in_split, const void *dev_out,
                                      void *host_out, size_t out_bytes, size_t out_split, photon_stream stream) {
    if (!ctx || !args) return PHOTON_ERR_INVALID_ARG;
    if ((in_bytes && (!host_in || !dev_in)) || (out_bytes && (!dev_out || !host_out))) return PHOTON_ERR_INVALID_ARG;
    if (in_split > in_bytes || out_split > out_bytes) return PHOTON_ERR_INVALID_ARG;
    const HostPlan hp{static_cast<const char *>(host_in), static_cast<char *>(dev_in), in_bytes, in_split,
                      static_cast<const char *>(dev_out), static_cast<char *>(host_out), out_bytes, out_split};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const photon_status s = step_impl(ctx, args, stream, &hp);
    if (s != PHOTON_OK) return s;
    // a step is tens of microseconds: poll for its end (a blocking wait pays a wake-up of several microseconds),
    // and hand over to the blocking wait when the stream turns out to hold much more work than that (how long to
    // poll is the context's: photon_set_host_step_tuning; 0 blocks at once)
    const auto t0 = std::chrono::steady_clock::now();
    cudaError_t e;
    while ((e = cudaStreamQuery(st)) == cudaErrorNotReady)
        if (std::chrono::steady_clock::now() - t0 >= std::chrono::microseconds(ctx->host_poll_us)) {
            e = cudaStreamSynchronize(st);
            break;
        }
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_device_status(photon_ctx *ctx, int32_t *bits_out, int32_t clear) {
    if (!ctx || !bits_out) return PHOTON_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return PHOTON_ERR_CUDA;
    if (cudaMemcpy(bits_out, ctx->status, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
        return PHOTON_ERR_CUDA;
    if (clear && cudaMemset(ctx->status, 0, sizeof(int32_t)) != cudaSuccess) return PHOTON_ERR_CUDA;
    // a kernel that gave up on a wait, or stopped at an index that was out of range, may have left arrival
    // tickets or counters behind (the hand-out counters of the whole-chunk attention, the readers' counter of
    // a folded-in append); they must read zero again
    if (clear && (*bits_out & (PHOTON_DEV_TIMEOUT | PHOTON_DEV_BAD_INDEX)) &&
        (cudaMemset(ctx->tickets, 0, ctx->n_tickets * sizeof(int32_t)) != cudaSuccess ||
         cudaMemset(ctx->work, 0, 32 * sizeof(int32_t)) != cudaSuccess))       // words 32..63 of the status block
        return PHOTON_ERR_CUDA;
    return PHOTON_OK;
}

photon_status photon_read_probe(photon_ctx *ctx, const void *src, size_t bytes, int32_t ctas, uint32_t *sum_out,
                                photon_stream stream) {
    if (!ctx || ctas < 0 || (bytes && !src) || !aligned16(src) || bytes % 16 != 0) return PHOTON_ERR_INVALID_ARG;
    const cudaError_t e = launch_read_probe(ctx, src, bytes, ctas, sum_out, static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

photon_status photon_wait_probe(photon_ctx *ctx, int64_t limit_ns, photon_stream stream) {
    if (!ctx || limit_ns < 0 || limit_ns > 100000000) return PHOTON_ERR_INVALID_ARG;       // a tenth of a second at most
    const cudaError_t e = launch_wait_probe(ctx, (unsigned long long)limit_ns, static_cast<cudaStream_t>(stream), &ctx->launches);
    return e == cudaSuccess ? PHOTON_OK : PHOTON_ERR_CUDA;
}

int64_t photon_launch_count(const photon_ctx *ctx) { return ctx ? ctx->launches : 0; }

photon_status photon_set_attention_ctas(photon_ctx *ctx, int32_t n) {
    if (!ctx || n < 0) return PHOTON_ERR_INVALID_ARG;
    ctx->attn_ctas = (n <= 0 || n > ctx->max_ctas) ? 0 : n;
    return PHOTON_OK;
}

photon_status photon_set_host_step_tuning(photon_ctx *ctx, int64_t pause_ns, int64_t poll_us) {
    if (!ctx || pause_ns < 0 || pause_ns > 1000000 || poll_us < 0 || poll_us > 10000000) return PHOTON_ERR_INVALID_ARG;
    ctx->host_pause_ns = pause_ns;
    ctx->host_poll_us = poll_us;
    return PHOTON_OK;
}

const char *photon_status_str(photon_status s) {
    switch (s) {
        case PHOTON_OK: return "ok";
        case PHOTON_ERR_INVALID_ARG: return "invalid argument";
        case PHOTON_ERR_UNSUPPORTED: return "unsupported shape or device";
        case PHOTON_ERR_CUDA: return "CUDA runtime error";
        case PHOTON_ERR_WORKSPACE: return "workspace too small for this call";
    }
    return "unknown status";
}

}  // extern "C"
