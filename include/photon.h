/* photon.h - C boundary of the PHOTON decode-step library (sm_100a).
 *
 * One recursive-generation step of PHOTON (Section 2.3.3): the coarsest
 * stream appends one latent to its KV cache and attends over it (the
 * attention and cache halves of STEP, Eq. 12 / Eq. 13), the context converter
 * expands the resulting latent into P prefix vectors (Section 2.1.2), and the
 * local decoders run bounded causal attention over P prefix rows plus at most
 * C in-chunk rows, independently for every in-flight chunk (Eq. 6-7).
 *
 * Conventions that hold for every call
 *  - All tensor pointers are DEVICE pointers owned by the caller, 16-byte
 *    aligned, bf16 stored as raw uint16 bits, C order.  The library owns only
 *    the photon_ctx (split-K workspace and a 4-byte device status word).
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and
 *    return at once; nothing synchronises except photon_device_status.
 *  - The return value reports host-side problems only (bad arguments, a
 *    failed launch).  Nothing is launched when it is not PHOTON_OK.
 *  - Device-side anomalies never trap.  They set bits in the status word:
 *    an append without room writes nothing (PHOTON_DEV_CAPACITY); an
 *    out-of-range unit id, slot or shared id skips that item and zero-fills
 *    its output row (PHOTON_DEV_BAD_INDEX); a bounded wait that ran out
 *    (PHOTON_DEV_TIMEOUT) leaves the affected outputs undefined.
 *  - q and k arrive already position-encoded; the library applies no rotary
 *    or other positional transform.
 *  - There is no CPU fallback: without a CUDA device photon_create fails.
 *  - Host threads: the library keeps a little host-side state (tensor-map
 *    caches, per-kernel launch attributes) that it does not lock.  Calls on
 *    one context, and calls of photon_coarse_attn_noalloc on one device, must
 *    not run concurrently with each other or with calls on another context;
 *    a caller with several threads serialises its calls into the library.
 *  - len, slot, shared_id and page_table must not change while a call that
 *    reads them is in flight on the device (a kernel of the caller's that
 *    writes them belongs before the call in the same stream).
 */
#ifndef PHOTON_H
#define PHOTON_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t photon_bf16;            /* raw bf16 bits */
typedef struct photon_ctx photon_ctx;
typedef void *photon_stream;             /* cudaStream_t */
typedef void *photon_event;              /* cudaEvent_t  */

typedef enum {
  PHOTON_OK = 0,
  PHOTON_ERR_INVALID_ARG = 1,            /* NULL / misaligned pointer, size out of range */
  PHOTON_ERR_UNSUPPORTED = 2,            /* shape the kernels are not built for */
  PHOTON_ERR_CUDA = 3,                   /* a CUDA runtime call or launch failed */
  PHOTON_ERR_WORKSPACE = 4               /* call needs more workspace than the ctx was created with */
} photon_status;

enum {                                   /* device status bits */
  PHOTON_DEV_CAPACITY = 1,
  PHOTON_DEV_BAD_INDEX = 2,
  PHOTON_DEV_TIMEOUT = 4
};

enum {                                   /* storage order of the converter weight */
  PHOTON_W_IN_MAJOR = 0,                 /* W[k][n]: [D, P*D], row k = input feature   */
  PHOTON_W_OUT_MAJOR = 1                 /* W[n][k]: [P*D, D], row n = output column (the order of a
                                            kernel-size-1 convolution weight)          */
};

/* Model shape, fixed per context.  Hq query heads share Hkv KV heads in
 * contiguous groups (query head h reads KV head h / (Hq/Hkv)).  dh must be 64
 * or 128, Hq/Hkv at most 16, D = d_model a multiple of 64, P + C at most 64.
 * max_queries: largest number of queries (sequences, branches or chunks) any
 * single attention call will carry; max_splits: upper bound on the number of
 * key ranges a shared prefix is split into (0 = library default; at most 8
 * are used).  max_queries sizes the workspace. */
typedef struct {
  int32_t Hq, Hkv, dh, D, P, C;
  int32_t max_queries;
  int32_t max_splits;
} photon_config;

/* A KV cache: coarse (one unit per sequence), token-level (for
 * photon_flat_attn) or chunk-local (one unit per chunk buffer, cap = P + C).
 *   k, v        [n_units, Hkv, cap, dh]; rows [0, len[u]) of unit u are valid,
 *               rows beyond may hold anything (including NaN bit patterns)
 *               and never influence a result.
 *   len         [n_units] device int32.
 *   max_len     host-side upper bound on every len[u] during the call
 *               (0 = cap).  It steers how many CTAs are launched and, for a
 *               cache with shared prefixes, whether the units' own rows are
 *               read by the shared-prefix kernel itself (at most 32 of them
 *               per unit: one launch) or by a second kernel.  It has to hold:
 *               a unit longer than max_len may have the rows beyond it
 *               ignored, with PHOTON_DEV_BAD_INDEX set.
 * Optional shared prefixes (Section 1: long-context, multi-query serving; one
 * document, many query branches): unit u with shared_id[u] = s >= 0 attends
 * rows [0, shared_len[s]) of segment s followed by its own rows, exactly as
 * if the prefix had been copied in front of its cache; the prefix is stored
 * and read once.  k_shared = NULL disables this.
 *   k_shared, v_shared [n_shared, Hkv, cap_shared, dh]; shared_len [n_shared];
 *   shared_id [n_units], -1 = none; max_shared_len like max_len.
 * Optional paging (a serving layout; the paper has no counterpart): with
 * page_table != NULL, k and v are pools [n_pages, Hkv, page_rows, dh] and row r
 * of unit u lives in page page_table[u * pages_per_unit + r / page_rows] at row
 * r % page_rows; cap must equal pages_per_unit * page_rows and page_rows must
 * be a multiple of 64.  Pages of different units must be distinct.  A page id
 * outside [0, n_pages) sets PHOTON_DEV_BAD_INDEX (page 0 is read instead; an
 * append is dropped).  Accepted by photon_kv_append, photon_coarse_attn,
 * photon_flat_attn and what is built on them; the chunk-local calls and the
 * no-allocation call take contiguous caches only (INVALID_ARG). */
typedef struct {
  photon_bf16 *k, *v;
  int32_t *len;
  int32_t n_units, cap, max_len;
  const photon_bf16 *k_shared, *v_shared;
  const int32_t *shared_len, *shared_id;
  int32_t n_shared, cap_shared, max_shared_len;
  const int32_t *page_table;             /* [n_units, pages_per_unit] device int32, or NULL */
  int32_t page_rows, pages_per_unit, n_pages;
} photon_kv;

/* Creates a context on the current CUDA device: validates cfg, allocates the
 * split-K workspace and the status word.  The only allocating call besides
 * photon_destroy's frees.  *out is NULL on failure. */
photon_status photon_create(photon_ctx **out, const photon_config *cfg);
photon_status photon_destroy(photon_ctx *ctx);

/* Cache half of the streaming update STEP (Eq. 12, Eq. 13): KV_{<=g} is
 * KV_{<=g-1} plus the new unit's K and V.  Item i (i < n) writes n_rows rows
 * k_new, v_new [n, n_rows, Hkv, dh] into unit u = unit_ids ? unit_ids[i] : i
 * at rows len[u] .. len[u]+n_rows-1 and adds n_rows to len[u].  A bit copy.
 * Unit ids within one call must be distinct.  With n_rows = P the same call
 * installs a chunk's prefix rows; with n_rows = 1 it appends an in-chunk row
 * (chunk-local caches are discarded at chunk boundaries by resetting len,
 * Section 2.3.3).  No room: nothing written, PHOTON_DEV_CAPACITY. */
photon_status photon_kv_append(photon_ctx *ctx, photon_kv *cache, const photon_bf16 *k_new,
                               const photon_bf16 *v_new, const int32_t *unit_ids, int32_t n,
                               int32_t n_rows, photon_stream stream);

/* Attention half of STEP for the coarsest stream (Eq. 12; causal Transformer
 * F^(L) of Section 2.1.1 whose cache holds T / C_{<=L} units, Section 2.3.3):
 * for unit u and query head h,
 *   s_i = scale * <q[u,h], K[u,h/G,i]>,  i over the shared prefix rows (if any)
 *   then rows [0, len[u]);  out[u,h] = sum_i softmax(s)_i V[u,h/G,i].
 * For the newest position the causal mask selects exactly the valid rows, so
 * a caller appends first and then attends.  q, out: [n_units, Hq, dh] bf16;
 * lse: [n_units, Hq] float (log-sum-exp of the logits, natural log) or NULL.
 * No valid key: out row = 0, lse = -inf.  fp32 accumulation, one rounding to
 * bf16 at the output.  The keys of all units are dealt out evenly over a
 * persistent grid; a cache cut by a grid boundary is merged by log-sum-exp in
 * a fixed order, so a call is deterministic, while the last bits of a unit's
 * result may depend on where in the batch it sits.  A shared prefix is read
 * once for all its branches. */
photon_status photon_coarse_attn(photon_ctx *ctx, const photon_kv *cache, const photon_bf16 *q,
                                 photon_bf16 *out, float *lse, float scale, photon_stream stream);

/* The same operation on a token-level cache (what a flat Transformer reads
 * per generated token, Section 2.3.1); exists to report KV bytes per token
 * of the flat baseline next to the coarse stream's. */
photon_status photon_flat_attn(photon_ctx *ctx, const photon_kv *cache, const photon_bf16 *q,
                               photon_bf16 *out, float *lse, float scale, photon_stream stream);

/* Context converter U^(l) (Section 2.1.2): one latent -> P conditioning
 * vectors, U[b, r, j] = sum_k x[b,k] * W[k, r*D + j] (+ bias[r*D + j]).
 * x [B, D]; w in the order given by w_layout; bias [P*D] or NULL;
 * U [B, P, D]; all bf16, fp32 accumulation, one rounding at the output. */
photon_status photon_converter(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *w,
                               int32_t w_layout, const photon_bf16 *bias, photon_bf16 *U, int32_t B,
                               photon_stream stream);

/* The two halves of the top-level context chunker C^(L) (Section 2.1.1; step
 * (ii) of a recursive-generation step, Section 2.3.3: the C_L reconstructed
 * lower-level latents of the meta-context just decoded are concatenated and
 * summarised into the next input of the top-level encoder).  The parameter
 * tables of Appendix B size it as a scale per concatenated feature, a weight
 * [C_L * D, D] and a bias.
 *
 * photon_rmsnorm: out[r, c] = x[r, c] * gamma[c] / sqrt(mean_c x[r, c]^2 + eps),
 * x, out [rows, cols] bf16 (out may alias x), gamma [cols] or NULL (ones),
 * cols a multiple of 8, eps >= 0; fp32 sums, one rounding to bf16.
 *
 * photon_linear: y[b, n] = sum_k x[b, k] * W[k, n] (+ bias[n]) (+ residual[b, n]);
 * x [B, K], w in the order given by w_layout ([K, N] or [N, K]), bias [N] or
 * NULL, residual [B, N] or NULL (may alias y), y [B, N]; K and N multiples of
 * 64 (else INVALID_ARG); bf16 in, fp32 accumulation on the tensor cores, one
 * rounding at the output; deterministic.  The converter is the case K = D,
 * N = P * D.  All pointers device, 16-byte aligned, owned by the caller; one
 * kernel each on `stream`, no workspace. */
photon_status photon_rmsnorm(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *gamma, float eps,
                             photon_bf16 *out, int32_t rows, int32_t cols, photon_stream stream);
photon_status photon_linear(photon_ctx *ctx, const photon_bf16 *x, const photon_bf16 *w, int32_t w_layout,
                            const photon_bf16 *bias, const photon_bf16 *residual, photon_bf16 *y, int32_t B,
                            int32_t K, int32_t N, photon_stream stream);

/* The rest of one LLaMA layer of the top-level context encoder around the
 * attention of STEP (Eq. 12 / Eq. 13; Section 3.1: every model is a LLaMA
 * Transformer).  The paper fixes neither the rotary convention nor its base:
 * the half-split pairing (feature j with j + dh/2) and the base `theta` given
 * by the caller (10000 in the LLaMA reference) are used.
 *
 * photon_rope_split: qkv [n, (Hq + 2 Hkv) dh], the fused projection of n new
 * latents, is taken apart into q [n, Hq, dh], k [n, Hkv, dh], v [n, Hkv, dh]
 * (what photon_kv_append and photon_coarse_attn read); every head of q and k
 * is rotated by the item's position pos[i] (device int32; for a decode step
 * the cache length before the append).  Heads are those of the context.
 *
 * photon_swiglu: out[i, f] = silu(gu[i, f]) * gu[i, F + f]; gu [n, 2F], out
 * [n, F], F a multiple of 8.
 *
 * photon_encoder_step: the whole layer for the newest latent of every
 * sequence, nine kernels on `stream`: normalise x (g1) -> wqkv -> rope_split
 * at position len[b], which here writes k and v straight into row len[b] of
 * `cache` and sets len += 1 (contiguous or paged; the checks and status bits
 * of photon_kv_append; scratch->k_new and v_new stay unwritten) -> attention
 * over the grown cache -> wo + x -> normalise (g2) -> wgu -> swiglu -> wdown + h.
 * x, y [B, D] with B = cache->n_units and D = Hq * dh of the context;
 * weights in the order w_layout names: wqkv [D, (Hq + 2 Hkv) dh], wo [Hq dh,
 * D], wgu [D, 2F], wdown [F, D]; g1, g2 [D].  F a multiple of 64.  The
 * caller owns the intermediates in `scratch` (sizes beside the fields); each
 * is rounded to bf16 where the next kernel reads it.  y may alias x.  Where
 * the gate/up projection's slabs of 64 features occupy at least half of the
 * GPU's SMs (F / 64 slabs per 128 rows), and with thousands of rows, that
 * projection and the activation are one launch and scratch->gu is left
 * unwritten (eight launches); both projections are rounded to bf16 before
 * the activation either way.
 *
 * photon_decoder_step: the same layer of a local decoder G^(l) (Eq. 6-7) for
 * the newest in-chunk position of every in-flight chunk: `chunks` holds the
 * chunk buffers (cap <= P + C; x, y [n_units, D]), the position is the
 * buffer's length before the append (prefix rows count), and the attention
 * is the bounded one of photon_chunk_attn.
 *
 * photon_decoder_prefill: the same layer over a fresh converter prefix, the
 * first R_l positions of the sequence [U ; X_<j] of Eq. 6: U [n, P, D] (what
 * photon_converter wrote for n chunks) -> the P rows of item i are encoded at
 * positions 0..P-1, their key/value rows become rows 0..P-1 of chunk buffer
 * unit_ids[i] (or i; the buffer must be empty: len = 0, as after a chunk
 * boundary) and they attend causally among themselves
 * (photon_chunk_causal_attn); y [n, P, D].  `scratch` is sized for n * P rows.
 * With this call the converter's output reaches the chunk buffers that
 * photon_chunk_attn and photon_decoder_step read. */
typedef struct photon_layer {
  const photon_bf16 *g1, *wqkv, *wo, *g2, *wgu, *wdown;
  int32_t w_layout;          /* PHOTON_W_IN_MAJOR or PHOTON_W_OUT_MAJOR, all four weights */
  int32_t F;                 /* width of the MLP */
  float eps;                 /* of both normalisations */
  float theta;               /* rotary base */
} photon_layer;
typedef struct photon_layer_scratch {
  photon_bf16 *n;            /* [B, D]   normalised input of either half */
  photon_bf16 *qkv;          /* [B, (Hq + 2 Hkv) dh] */
  photon_bf16 *q;            /* [B, Hq, dh] */
  photon_bf16 *k_new, *v_new;/* [B, Hkv, dh]  written by photon_decoder_prefill only */
  photon_bf16 *att;          /* [B, Hq, dh] */
  photon_bf16 *h;            /* [B, D]   after the attention half */
  photon_bf16 *gu;           /* [B, 2F] */
  photon_bf16 *act;          /* [B, F] */
} photon_layer_scratch;
photon_status photon_rope_split(photon_ctx *ctx, const photon_bf16 *qkv, const int32_t *pos, int32_t n,
                                float theta, photon_bf16 *q, photon_bf16 *k, photon_bf16 *v,
                                photon_stream stream);
photon_status photon_swiglu(photon_ctx *ctx, const photon_bf16 *gu, photon_bf16 *out, int32_t n, int32_t F,
                            photon_stream stream);
photon_status photon_encoder_step(photon_ctx *ctx, const photon_layer *layer, const photon_layer_scratch *scratch,
                                  const photon_bf16 *x, photon_kv *cache, photon_bf16 *y, float scale,
                                  photon_stream stream);
photon_status photon_decoder_step(photon_ctx *ctx, const photon_layer *layer, const photon_layer_scratch *scratch,
                                  const photon_bf16 *x, photon_kv *chunks, photon_bf16 *y, float scale,
                                  photon_stream stream);
photon_status photon_decoder_prefill(photon_ctx *ctx, const photon_layer *layer, const photon_layer_scratch *scratch,
                                     const photon_bf16 *U, photon_kv *chunks, const int32_t *unit_ids, int32_t n,
                                     photon_bf16 *y, float scale, photon_stream stream);

/* Bounded causal attention of the local decoders G^(l) (Eq. 6-7): query c
 * (q [Nc, Hq, dh]) attends rows [0, len[u]) of chunk buffer u = slot ?
 * slot[c] : c of `chunks` (cap = P + C; rows 0..P-1 the converter prefix,
 * rows P.. the in-chunk positions written so far) and nothing else, so the
 * span is bounded by P + C whatever the context length.  out [Nc, Hq, dh].
 * Shared-prefix fields of `chunks` must be unset. */
photon_status photon_chunk_attn(photon_ctx *ctx, const photon_kv *chunks, const photon_bf16 *q,
                                const int32_t *slot, photon_bf16 *out, int32_t Nc, float scale,
                                photon_stream stream);

/* The local decoder's attention at `rows` consecutive positions of every
 * chunk at once: the teacher-forced form of Eq. 6 (all positions of a chunk in
 * one pass, or the P-row pass over a fresh converter prefix) under the
 * standard causal mask described below Eq. 7.  Query t of chunk c (q [Nc,
 * rows, Hq, dh]) stands at row row0 + t of chunk buffer u = slot ? slot[c] : c
 * and attends rows 0 .. row0 + t of that buffer and nothing else.  A position
 * at or beyond len[u] does not exist yet: its output row is zero.  out [Nc,
 * rows, Hq, dh], bf16, written in full.  Requires cap <= min(P + C, 64),
 * row0 >= 0, rows >= 1, row0 + rows <= cap (else INVALID_ARG); q and out are
 * device pointers, 16-byte aligned, owned by the caller; a slot outside
 * [0, n_units) gives zero rows and sets PHOTON_DEV_BAD_INDEX.  One kernel on
 * `stream`, no workspace.  Shared-prefix fields of `chunks` must be unset. */
photon_status photon_chunk_causal_attn(photon_ctx *ctx, const photon_kv *chunks, const photon_bf16 *q,
                                       const int32_t *slot, photon_bf16 *out, int32_t Nc, int32_t row0,
                                       int32_t rows, float scale, photon_stream stream);

/* One decode step on one stream, in the order of Section 2.3.3: append
 * (k_new, v_new) to `coarse`; coarse attention of q_coarse over the grown
 * cache -> out_coarse (lse_coarse optional); converter on x, or, when x is
 * NULL, on out_coarse viewed as [B, Hq*dh] (requires Hq*dh == D and
 * B == coarse->n_units); chunk attention of q_chunk over `chunks`.
 * ev_attn_begin / ev_attn_end, when not NULL, are recorded on the stream
 * around the coarse attention launches (for timing that part in place).
 * For the caller everything is ordered on `stream`.  Inside, a small chunk
 * workload runs beside the other parts on a low-priority stream of the
 * context that forks from `stream` when the call starts and joins it before
 * the call's work ends (it shares no data with them).  A context serves one
 * stream at a time: its workspace, tickets and this side stream are not
 * meant for concurrent calls. */
typedef struct {
  photon_kv *coarse;
  const photon_bf16 *k_new, *v_new, *q_coarse;
  photon_bf16 *out_coarse;
  float *lse_coarse;
  float scale_coarse;
  const photon_bf16 *x, *w, *bias;
  int32_t w_layout;
  photon_bf16 *U;
  int32_t B;
  const photon_kv *chunks;
  const photon_bf16 *q_chunk;
  const int32_t *slot;
  photon_bf16 *out_chunk;
  int32_t Nc;
  float scale_chunk;
  photon_event ev_attn_begin, ev_attn_end;
} photon_step_args;

photon_status photon_decode_step(photon_ctx *ctx, const photon_step_args *args, photon_stream stream);

/* The same step for a caller whose inputs and results live in HOST memory
 * (the serving loop around Section 2.3.3: what a step consumes arrives from the
 * host, what it produces goes back).  in_bytes travel from host_in to dev_in,
 * the step runs, out_bytes travel from dev_out to host_out, and the call waits
 * for `stream`; when it returns PHOTON_OK host_out holds the results.
 *   host_in, host_out  host pointers owned by the caller; page-locked memory
 *                      makes the copies asynchronous to the host, pageable
 *                      memory works and is staged by the driver.
 *   dev_in, dev_out    device staging areas owned by the caller: the input
 *                      pointers of `args` (k_new, v_new, queries, lengths ...)
 *                      point into dev_in and its output pointers into dev_out;
 *                      the call only moves the bytes.  Either size may be 0.
 *   in_split           bytes [0, in_split) of the input are what the append,
 *                      the coarse attention and the converter read; the rest is
 *                      read by the chunk attention only (q_chunk, slot).
 *   out_split          bytes [0, out_split) of the output are written by the
 *                      coarse attention (out_coarse, lse_coarse) and, when the
 *                      caller wants it on the host, by the converter (U, which
 *                      then comes after the coarse attention's arrays: what
 *                      precedes U leaves beside the converter, U and what
 *                      follows it after the converter); the rest by the chunk
 *                      attention (out_chunk).
 * With in_split == in_bytes and out_split == out_bytes everything is copied in
 * before the step and out after it.  Otherwise, when the chunk attention runs
 * on the context's side stream (see photon_decode_step), the two parts of a
 * buffer travel apart: the chunk attention's inputs cross the bus while the
 * append and the coarse attention already run, its results leave when it ends,
 * and the coarse results leave beside the converter.  Where both host buffers
 * are page-locked memory that the device can address and q_chunk, slot and
 * out_chunk lie wholly in the chunk attention's halves of the staging areas,
 * the chunk attention reads and writes the host buffers themselves when it runs
 * in line, or beside the coarse part with at most 1 MiB each way (the same bytes cross the bus, no copy is enqueued
 * for them, the coarse results still leave beside the converter) and those
 * halves of the staging areas are left untouched.  A buffer laid out
 * otherwise than declared gives stale inputs or results: the call cannot tell.
 * NULL ctx or args, a NULL pointer beside a non-zero size, or a split beyond
 * its size: INVALID_ARG, nothing is enqueued.  An error of the step itself is
 * returned without waiting; the stream is then left as the step left it. */
photon_status photon_decode_step_host(photon_ctx *ctx, const photon_step_args *args, const void *host_in,
                                      void *dev_in, size_t in_bytes, size_t in_split, const void *dev_out,
                                      void *host_out, size_t out_bytes, size_t out_split, photon_stream stream);

/* Two host-side habits of photon_decode_step_host, both found by measurement on
 * one machine and therefore adjustable per context: pause_ns (default 1500, at
 * most 1e6, 0 = none) is how long the call waits between enqueuing its first
 * host-to-device copy and its first kernel launch (launches that follow the
 * copy within a microsecond made the whole step end later there); poll_us
 * (default 2000, at most 1e7, 0 = block at once) is how long the call polls
 * the stream for the step's end before it falls back to a blocking wait.
 * Neither changes what the step computes. */
photon_status photon_set_host_step_tuning(photon_ctx *ctx, int64_t pause_ns, int64_t poll_us);

/* Reads (and optionally clears) the device status word.  Synchronises the
 * whole device; the only call that does.  Clearing a PHOTON_DEV_TIMEOUT or a
 * PHOTON_DEV_BAD_INDEX also puts the context's arrival tickets back to zero,
 * so the context stays usable after a kernel that gave up on a wait or
 * stopped at an index out of range. */
photon_status photon_device_status(photon_ctx *ctx, int32_t *bits_out, int32_t clear);

/* The paper has no counterpart to this call: it exists for hosts that must not
 * allocate device memory (a serving process whose memory pool owns the whole
 * device, a thread that may not take the allocator's locks or its implicit
 * synchronisation, a process that has promised a fixed footprint), where
 * photon_create is unusable.  It computes what photon_coarse_attn computes,
 * for a cache without shared prefixes, and needs no context: the kernel's
 * workspace is an array inside the library image (about 5.4 MB per GPU that
 * loads the library, held until the process exits).  Nothing here calls
 * cudaMalloc, cudaFree or an allocating library routine.
 *   cfg         only Hq, Hkv and dh are read.
 *   cache, q, out, lse, scale, stream   as for photon_coarse_attn.
 *   dev_status  device int32 the kernel ORs PHOTON_DEV_* bits into, or NULL
 *               (then they go to a word inside the array that nobody reads).
 * Limit: n_units * Hkv <= PHOTON_NOALLOC_MAX_STREAMS, else
 * PHOTON_ERR_WORKSPACE and nothing is launched; a shared prefix gives
 * PHOTON_ERR_UNSUPPORTED.  The first call on a device looks up the array's
 * device address; make that call before capturing a stream.  All calls on a
 * device share the array and the call clears the part that must start at
 * zero, so calls that overlap on one GPU race: keep them in stream order. */
#define PHOTON_NOALLOC_MAX_STREAMS 16384
photon_status photon_coarse_attn_noalloc(const photon_config *cfg, const photon_kv *cache,
                                         const photon_bf16 *q, photon_bf16 *out, float *lse, float scale,
                                         int32_t *dev_status, photon_stream stream);

/* Sets the persistent grid of photon_coarse_attn / photon_flat_attn to n CTAs
 * (0 or more than the device holds, two per SM: back to the default, where
 * the library picks a grid of at most 7/8 of what the device holds, lined up
 * with the number of (unit, KV head) streams of the call).  The keys of a call
 * are dealt out evenly over the grid, so n also moves the points where a long
 * cache is cut and merged by log-sum-exp; a smaller grid leaves SMs free for
 * work on another stream.  Takes effect from the next call. */
photon_status photon_set_attention_ctas(photon_ctx *ctx, int32_t n);

/* Two measurement and test aids without a counterpart in the paper; neither is
 * part of a decode step.
 *
 * photon_read_probe streams `bytes` (a multiple of 16) of device memory at the
 * 16-byte aligned pointer src into shared memory and computes nothing: same
 * launch, grid and ring of bulk copies as the coarse attention, so its time on
 * a buffer of the size an attention call reads is the ceiling that call can be
 * held against beside the HBM peak (tens of megabytes are bound by start-up
 * and drain, not by bandwidth).  ctas: the grid, 0 = the attention's default.
 * sum_out: device uint32 (or NULL) to which the kernel adds the sum, modulo
 * 2^32, of the first little-endian 32-bit word of every 128 bytes it read; the
 * caller clears it.  One kernel on `stream`.
 *
 * photon_wait_probe launches one thread that waits on a barrier nobody
 * arrives at, gives up after limit_ns nanoseconds (at most 1e8), sets
 * PHOTON_DEV_TIMEOUT, leaves one arrival ticket of the context non-zero (as a
 * kernel that stopped half way would) and returns by itself.  It exists so
 * that a test can see the path every bounded wait of the library takes when it
 * runs out, and that photon_device_status(clear) leaves the context usable. */
photon_status photon_read_probe(photon_ctx *ctx, const void *src, size_t bytes, int32_t ctas, uint32_t *sum_out,
                                photon_stream stream);
photon_status photon_wait_probe(photon_ctx *ctx, int64_t limit_ns, photon_stream stream);

/* Number of kernels the library has launched through this context so far. */
int64_t photon_launch_count(const photon_ctx *ctx);

const char *photon_status_str(photon_status s);

#ifdef __cplusplus
}
#endif
#endif /* PHOTON_H */
