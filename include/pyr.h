/*
 * pyr.h - C ABI of the PyramidInfer prefill-selection hot path for NVIDIA B200
 * (sm_100a).
 *
 * The library implements one layer-wise step of PyramidInfer (arXiv
 * 2405.12532, Algorithm 1, prefill branch, and the attention of the generation
 * phase of Section 4.1):
 *
 *   pyr_prefill_layer   attention weights over the tokens the layer received,
 *                       the attention output, and the ensemble score A_e that
 *                       the most recent L queries give every context key;
 *   pyr_select_compact  TopP index (a count-based top-k) + Gather: K/V of the
 *                       kept keys go to the layer's cache, rows that feed the
 *                       next layer are compacted in place;
 *   pyr_decode_attn     one generation step of one layer over its compressed,
 *                       per-layer-sized cache;
 *   pyr_cache_alloc     the pyramid itself: per-layer budgets from the ratio
 *                       schedule and the cache carved out of caller memory.
 *
 * Conventions
 *   - Plain C. Every call returns a pyr_status_t, never throws, aborts or
 *     prints.
 *   - Pointers marked "device" are caller-owned device memory that must stay
 *     valid until the stream work that uses them has finished. Pointers marked
 *     "host" are read (or written) before the call returns.
 *   - The library allocates no device memory: the caller passes one buffer of
 *     pyr_cache_bytes() bytes. Only the host-side handle is library-owned.
 *   - Every launching call takes a CUDA stream (cudaStream_t passed as void*,
 *     NULL = the default stream), enqueues its kernels there and returns; it
 *     does not synchronise. All shapes follow from the schedule on the host,
 *     so nothing is copied back.
 *   - A device-side wait that runs out (bounded spin on an mbarrier) records a
 *     code in a device status word and the kernel returns; read it with
 *     pyr_cache_status().
 *   - A handle is not thread-safe; use one per thread or lock around it.
 *
 * Tensor layouts (element = bf16 or fp32 as configured, D = head_dim innermost
 * and contiguous)
 *   q, out        [B, n, Hq,  D]   strides given in elements
 *   k, v          [B, n, Hkv, D]   strides given in elements
 *   layer cache   [B, Hkv, cap_l, D] for K and for V
 *   scores        [B, G, c]  fp32, G = sel_groups, c = n - L context keys
 *   lse           [B, Hq, n] fp32, natural log of the softmax denominator
 *   kept / pos    [B, G, n_out] int32
 */
#ifndef PYR_H_
#define PYR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PYR_OK = 0,
  PYR_ERR_INVALID = 1,          /* a value outside its documented range            */
  PYR_ERR_NULL = 2,             /* a required pointer is NULL                      */
  PYR_ERR_UNSUPPORTED = 3,      /* dtype / head_dim / size / device not supported  */
  PYR_ERR_BUFFER_TOO_SMALL = 4, /* dev_buf smaller than pyr_cache_bytes()          */
  PYR_ERR_CAPACITY = 5,         /* decode append beyond max_new_tokens             */
  PYR_ERR_ORDER = 6,            /* call out of the prefill/select/decode sequence  */
  PYR_ERR_CUDA = 7,             /* a CUDA runtime call failed                      */
  PYR_ERR_TIMEOUT = 8,          /* a bounded device-side wait ran out              */
  PYR_ERR_SCRATCH_LIMIT = 9,    /* problem exceeds the library's built-in scratch  */
  PYR_ERR_HOST_MEMORY = 10      /* the host-side handle could not be allocated     */
} pyr_status_t;

typedef enum { PYR_BF16 = 0, PYR_F32 = 1 } pyr_dtype_t;

/* flags */
#define PYR_FLAG_CUDA_CORE_PREFILL 1u /* bf16 prefill on the CUDA-core kernel (validation aid) */
#define PYR_FLAG_POS_REENCODE 4u      /* Appendix A.2, first choice: the kept tokens' positions are re-encoded from 0
                                         in order after every selection; default is the second choice (gather the
                                         original positions), which the paper finds slightly better */
#define PYR_FLAG_GEN_RESELECT 2u      /* keep each layer's recent queries so that pyr_decode_reselect can
                                         update the PvC during generation (Section 4.1, Generation Phase) */
#define PYR_FLAG_SELECT_FIRST 8u      /* select-first ordering (bf16, head_dim 128): pyr_prefill_layer computes the
                                         query tiles that hold the recent window, the scores and the selection
                                         first, then the remaining query tiles, writing each kept row of `out`
                                         straight to its place among the kept rows of its selection group (dropped
                                         rows are not written). pyr_select_compact then gathers K/V and, when its
                                         `rows` is that same `out`, only moves the rows of the first tiles down;
                                         any other `rows` is compacted in full as always. The results equal the
                                         default ordering's. Layers that drop nothing, and configurations the
                                         tensor-core kernels do not cover, take the default ordering. */

/*
 * Parameters of Algorithm 1 (recent window length L, minimum PvC lengths N_l,
 * ratio p and its decay, given here as one explicit ratio per layer) plus the
 * attention geometry.
 */
typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;      /* Hq                                                        */
  int32_t n_kv_heads;     /* Hkv, divides Hq                                           */
  int32_t head_dim;       /* D: 64 or 128. The tensor-core (tcgen05) prefill kernels are
                             built for bf16 with D = 128; bf16 with D = 64 and all of fp32
                             run on the CUDA-core kernels, far below tensor-core speed     */
  int32_t sel_groups;     /* G: 1 (one kept set per sequence) or Hkv (one per KV head) */
  int32_t dtype;          /* pyr_dtype_t of q/k/v/out and of the cache                 */
  int32_t batch;          /* B                                                         */
  int32_t prompt_len;     /* N, the same for every sequence of the batch               */
  int32_t recent_len;     /* L >= 1: the recent window S_r, never evicted              */
  int32_t max_new_tokens; /* T: rows reserved per layer for decode appends             */
  const double* ratio;    /* host [n_layers]: fraction of the ORIGINAL context
                             c_0 = N - L that layer l keeps; each in [0,1],
                             non-increasing                                            */
  const int32_t* min_len; /* host [n_layers] or NULL: N_l, lower bound on the kept
                             length (window included) of layer l. FIXED-COUNT MODE
                             (Section 4.1, last sentence: a fixed number of PvCs per layer,
                             "unlimited input like StreamingLLM"): ratio[l] = 0 and
                             min_len[l] = count_l + L keep exactly count_l context keys in
                             layer l; with pyr_decode_reselect every s <= T steps the cache
                             never exceeds count_l + L + s rows however long the generation */
  const float* recent_w;  /* host [L] or NULL: non-negative weights of the recent
                             queries, oldest first. NULL = linear ramp
                             2(i+1)/(L(L+1)), which sums to 1                          */
  float softmax_scale;    /* 0 = 1/sqrt(D)                                             */
  uint32_t flags;
} pyr_config_t;

typedef struct pyr_cache pyr_cache_t;

/* Algorithm 1's schedule (p, decay, N_l) as integers: for layer `layer` the
 * tokens it receives (n_in), the context keys it keeps (k_ctx; the kept length
 * is k_ctx + min(L, n_in)), the rows now in its cache (len_now) and the cache
 * capacity in rows (cap). k_ctx = min(c, max(floor(ratio*c_0), N_l - L, 0)).
 * Host arithmetic only; any out pointer may be NULL. */
pyr_status_t pyr_cache_layer_info(const pyr_cache_t* cache, int32_t layer, int32_t* n_in,
                                  int32_t* k_ctx, int32_t* len_now, int32_t* cap);

/* Size and alignment of the device buffer pyr_cache_alloc needs for `cfg`
 * (Section 4.1: each layer's cache holds only its PvC and window, plus T
 * decode rows; the buffer also holds scores (pooled, and per head for the
 * tensor-core score pass), lse, kept indices, positions, the decode workspace
 * and the status word). Validates cfg. */
pyr_status_t pyr_cache_bytes(const pyr_config_t* cfg, size_t* bytes, size_t* align);

/* Builds a cache handle over the caller's device buffer `dev_buf` (device,
 * `bytes` long, aligned as pyr_cache_bytes says). Copies cfg and its arrays.
 * Touches no device memory and makes no CUDA call. *out is set on PYR_OK. */
pyr_status_t pyr_cache_alloc(const pyr_config_t* cfg, void* dev_buf, size_t bytes,
                             pyr_cache_t** out);

/* Frees the host handle. The device buffer stays the caller's. */
pyr_status_t pyr_cache_free(pyr_cache_t* cache);

/* Starts a new prompt batch with the same configuration: layer 0's prefill is
 * expected next; clears the device status word on `stream`. */
pyr_status_t pyr_cache_reset(pyr_cache_t* cache, void* stream);

/* Device pointers (valid until the next pyr_select_compact) to the kept indices
 * [B, G, n_out] of `layer`'s selection - ascending positions within the layer's
 * input, window last - and to the ORIGINAL prompt positions of those tokens
 * (Appendix A.2, "gather" position encoding). `layer` must be the layer most
 * recently selected. */
pyr_status_t pyr_cache_kept(const pyr_cache_t* cache, int32_t layer, const int32_t** dev_idx,
                            const int32_t** dev_pos);

/* Device pointer to the pooled ensemble scores [B, G, c] that the most recent
 * pyr_prefill_layer(layer) wrote (valid until the next prefill call). */
pyr_status_t pyr_cache_scores(const pyr_cache_t* cache, int32_t layer, const float** dev_scores);

/* Device pointer to lse [B, Hq, n_in] of the most recent pyr_prefill_layer. */
pyr_status_t pyr_cache_lse(const pyr_cache_t* cache, int32_t layer, const float** dev_lse);

/* Device pointers to layer `layer`'s K and V cache [B, Hkv, cap, D]. */
pyr_status_t pyr_cache_kv(const pyr_cache_t* cache, int32_t layer, void** dev_k, void** dev_v);

/* Synchronises `stream`, copies the device status word to *host_status
 * (a pyr_status_t: PYR_OK or PYR_ERR_TIMEOUT) and returns it. */
pyr_status_t pyr_cache_status(pyr_cache_t* cache, void* stream, int32_t* host_status);

/*
 * Algorithm 1, "compute attention weights of KV" and
 * "A_e <- weighted_avg(A[-L:, :-L], dim=-2)" for one layer.
 *
 * q, k, v (device) hold the layer's n_in tokens in ascending original order.
 * Writes out = softmax(scale q k^T + causal mask) v for all n_in rows, lse into
 * the cache, and the pooled score
 *     score[b,g,j] = mean over the query heads h of group g of
 *                    sum_i w_i * A_h[c+i, j],   j < c = n_in - L,
 * into the cache. The L x c block of weights is never stored. Layers must be
 * called in order, each followed by pyr_select_compact (PYR_ERR_ORDER
 * otherwise). Strides are in elements; the innermost (D) stride is 1. For
 * bf16 the base pointers and strides must keep every row 16-byte aligned.
 */
pyr_status_t pyr_prefill_layer(pyr_cache_t* cache, int32_t layer, const void* q, const void* k,
                               const void* v, void* out, int64_t q_stride_b, int64_t q_stride_n,
                               int64_t q_stride_h, int64_t kv_stride_b, int64_t kv_stride_n,
                               int64_t kv_stride_h, int64_t o_stride_b, int64_t o_stride_n,
                               int64_t o_stride_h, void* stream);

/*
 * Algorithm 1, "TopP_index <- TopP(A_e, p)" and "PvC <- Gather(KV, TopP_index)".
 *
 * Per (sequence, selection group): the k_ctx largest scores left by
 * pyr_prefill_layer(layer) are kept, an exact tie going to the lower index;
 * the kept list is those keys in ascending order followed by the whole window.
 * K and V (device, the same tensors the prefill call read) are gathered into
 * the layer's cache. `rows` (device, may be NULL) is compacted IN PLACE to the
 * kept rows: row i of the result is former row kept[i]. With sel_groups == 1,
 * rows is [B, n_in, row_elems] (rows_stride_g must be 0), e.g. hidden states;
 * with sel_groups == Hkv it is addressed as
 * rows + b*rows_stride_b + g*rows_stride_g + i*rows_stride_n, row_elems
 * contiguous elements per row, e.g. the attention output of the group's heads.
 * Position ids are compacted alongside. *n_out (host, may be NULL) receives
 * k_ctx + window. Dropped rows are neither read nor written.
 */
pyr_status_t pyr_select_compact(pyr_cache_t* cache, int32_t layer, const void* k, const void* v,
                                int64_t kv_stride_b, int64_t kv_stride_n, int64_t kv_stride_h,
                                void* rows, int64_t row_elems, int64_t rows_stride_b,
                                int64_t rows_stride_n, int64_t rows_stride_g, int32_t* n_out,
                                void* stream);

/*
 * Section 4.1, generation phase: the new token's key and value (device,
 * [B, Hkv, D] contiguous) are appended to layer `layer`'s cache, then q
 * (device, [B, Hq, D] contiguous) attends over all len_now + 1 rows, unmasked.
 * out (device, [B, Hq, D]). Allowed once every layer has been selected.
 * PYR_ERR_CAPACITY when the layer already holds cap rows.
 */
pyr_status_t pyr_decode_attn(pyr_cache_t* cache, int32_t layer, const void* q, const void* k_new,
                             const void* v_new, void* out, void* stream);

/* Section 5.2, "Recent Sequence Ratio": the recent sequence S_r given as a fraction of the input
 * (the paper settles on 40 %). Returns the window length for pyr_config_t.recent_len:
 * floor(ratio * prompt_len) clamped to [1, prompt_len]; 0 for a negative ratio or an empty prompt.
 * Host arithmetic only. */
int32_t pyr_recent_len_from_ratio(int32_t prompt_len, double ratio);

/*
 * (No counterpart in the paper: a test aid for the failure path of the bounded device-side
 * waits.) Arms the cache so that the NEXT pyr_decode_attn call's loader thread leaves the first
 * chunk of cache rows of every split out and every wait of that launch spins a few thousand times
 * at most: the consumers' waits run out, the kernel returns without faulting or hanging,
 * pyr_cache_status reports PYR_ERR_TIMEOUT and `out` of that call is undefined. The call after it
 * is normal again; pyr_cache_reset clears the recorded status. Only the CUDA-core decode kernel
 * (fewer than 4 query heads per KV head, or fp32) honours it.
 */
pyr_status_t pyr_cache_arm_wait_test(pyr_cache_t* cache);

/*
 * Section 4.1, Generation Phase, and Algorithm 1's branch for a cache that
 * already holds past PvC: the recent window has slid over the generated tokens,
 * and the layer's PvC is selected again "the same as the prefill phase". The
 * attention weights of the window's queries (the last min(L, tokens so far)
 * tokens; query i sees the context rows and the window rows up to its own) are
 * taken over the layer's cache as it is now; their weighted average scores the
 * context rows (all rows before the window), pooled per selection group; the
 * layer's budget k_ctx of them is kept, ties to the lower row, and the cache's
 * K and V rows are compacted in place, in order, the window last. The cache then
 * holds k_ctx + window rows again: called every s decode steps it keeps a fixed
 * number of PvCs per layer, so T only has to cover s steps.
 * Nothing happens (and nothing is launched) while the context is not longer than
 * k_ctx. *c_ctx (may be NULL) receives the number of context rows scored, *n_out
 * (may be NULL) the rows the cache holds afterwards. pyr_cache_kept(layer) then
 * gives the kept row indices [B, G, n_out] into the cache as it was (its position
 * pointer repeats them: original positions are not tracked through generation)
 * and pyr_cache_scores(layer) the pooled scores [B, G, c_ctx].
 * Needs PYR_FLAG_GEN_RESELECT in the configuration (else PYR_ERR_UNSUPPORTED),
 * which reserves a ring of L + max(T, 1) query rows per layer and makes
 * pyr_prefill_layer (whose q rows must then be contiguous: strides Hq*D, D) and
 * pyr_decode_attn record their queries. Allowed once every layer has been selected.
 */
pyr_status_t pyr_decode_reselect(pyr_cache_t* cache, int32_t layer, int32_t* c_ctx, int32_t* n_out,
                                 void* stream);

/*
 * Decode attention for callers that must not allocate device memory.
 * (No counterpart in the paper: this is a packaging variant of pyr_decode_attn.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they
 * decode: code running inside a serving engine that has handed all device
 * memory to its own pool, plugins that are only given tensors, code on a
 * latency path where an allocation (an implicit device synchronisation) is not
 * acceptable. pyr_decode_attn needs a cache handle whose buffer includes a
 * split-K workspace; this entry point needs neither. The caller passes only
 * inputs and outputs:
 *   q [B, Hq, D], k_new / v_new [B, Hkv, D], out [B, Hq, D]      (device, contiguous)
 *   k_cache / v_cache [B, Hkv, cap, D] with rows 0..len-1 filled (device)
 * The new row is stored at row `len` of both caches and q attends over rows
 * 0..len, exactly as pyr_decode_attn does; the caller advances `len` itself.
 * softmax_scale 0 means 1/sqrt(D).
 *
 * The split-K partial results go to an array compiled into the library
 * (4 MiB per GPU, resident on every GPU that loads the library until the
 * process exits). A call whose B * Hq * splits * (D + 2) floats exceed it
 * returns PYR_ERR_SCRATCH_LIMIT and launches nothing. The split count is the
 * one pyr_decode_attn uses: min(64, floor(2 * SMs / (B * Hkv)),
 * ceil((len + 1) / 128)), at least 1, and then ceil((len + 1) / rows per
 * split) with the rows per split rounded up to a multiple of 16; with one
 * split no scratch is used at all.
 * All calls on a GPU share that array and it keeps the previous call's
 * contents (every slot is rewritten before it is read, so none needs
 * clearing): two calls whose kernels can overlap on the GPU - different
 * streams, or different threads - race on it; keep them on one stream or
 * order them with events. The first call on each GPU, whatever its sizes,
 * looks the array's device address up, which is a CUDA runtime call outside
 * the stream: make that first call before any stream capture begins. No
 * cudaMalloc, cudaFree or other allocating routine is called, on any call.
 * A bounded device-side wait that runs out is recorded in a word beside the
 * array; pyr_decode_attn_noalloc_status reads it. `out` of a call that hit one
 * is undefined.
 */
pyr_status_t pyr_decode_attn_noalloc(const void* q, const void* k_new, const void* v_new, void* out,
                                     void* k_cache, void* v_cache, int32_t batch, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t head_dim, int32_t dtype, int32_t len,
                                     int32_t cap, float softmax_scale, void* stream);

/*
 * (No counterpart in the paper.) Synchronises `stream`, then reports whether any
 * pyr_decode_attn_noalloc call on the current GPU recorded a device-side wait
 * that ran out since the last report: *host_status is 0 or PYR_ERR_TIMEOUT, and
 * the return value says the same. Reading clears the record. Allocates nothing.
 */
pyr_status_t pyr_decode_attn_noalloc_status(void* stream, int32_t* host_status);

/*
 * Decoder glue for whole-model workloads. (No counterpart in the paper beyond Appendix A.2's
 * choice of positions: these are the public Llama block's steps around the pyramid path, so that a
 * model can run end to end on this library's kernels. fp32 arithmetic for fp32 or bf16 storage;
 * dtype is a pyr_dtype_t. CUDA-core kernels, except the bf16 linear layer, see below.) All pointers
 * are device pointers, tensors row-major and contiguous, every call asynchronous on `stream`.
 *   embed   out[t, :] = table[ids[t], :]; table [vocab, d]. An id outside [0, vocab) zeroes its row
 *           and, if dev_status (a device int, may be NULL) is given, records PYR_ERR_INVALID in it.
 *   rmsnorm out = x / sqrt(mean(x^2) + eps) * gain; x, out [tokens, d] (may alias), gain [d].
 *   linear  y[m, n] = x[m, k] . w[n, k] (+ residual[m, n] if not NULL); w is [n, k] ("out, in").
 *           y may alias residual, not x. bf16 with 16-byte aligned pointers and k a multiple of 64
 *           runs on tensor cores (fp32 accumulation, one rounding to bf16 at the end): for m <= 64
 *           and n a multiple of 128 a weight-streaming kernel whose clusters split k and add their
 *           partial sums in a fixed order, else a tiled kernel (n a multiple of 8). Results are
 *           bit-reproducible run to run in every case. Everything else takes the CUDA-core kernel.
 *   rmsnorm_rows / linear_rows  the same two operations reading through a list of rows per sequence,
 *           so that kept rows are used where they lie and the hidden states are never compacted:
 *           rmsnorm_rows: out[b, i, :] = rmsnorm(x[b, rows[b * rows_stride + i], :]) for x [batch, n_src, d],
 *           out [batch, n_dst, d]; linear_rows: y[b, i, :] = x[b, i, :] . w^T + residual[b, res_rows[b *
 *           rows_stride + i], :] for x [batch, n_dst, k], residual [batch, n_src, n], y [batch, n_dst, n].
 *           The lists are device int32 (pyr_cache_kept's first pointer, a dense [B, n_out] array when
 *           sel_groups == 1: rows_stride = n_out); their entries must lie in [0, n_src), which is not checked.
 *   linear_split  the product of x [m, k] with a weight [n_parts * part_n, k] of up to four stacked
 *           projections (say q, k and v), part i written to its own tensor ys[i] [m, part_n] (ys: host
 *           array of device pointers): for at most 64 rows of x in bf16 the weight streams through one
 *           launch instead of one per projection; otherwise it is one product per part.
 *   linear_swiglu  out[m, n] = silu(x . w_gate^T) * (x . w_up^T), w_gate and w_up [n, k]: the gated MLP's
 *           first half in one pass, neither projection written out (fp32 accumulators go straight
 *           into the product). bf16 with 16-byte aligned pointers, k a multiple of 64 and n a
 *           multiple of 8 only; PYR_ERR_UNSUPPORTED otherwise (call linear twice and swiglu).
 *   rope    rotates, in place, the pairs (i, i + head_dim/2) of every head of x [tokens, n_heads,
 *           head_dim] by pos[t] * 10000^(-2i/head_dim): Appendix A.2's "gather" when pos holds the
 *           tokens' original positions (pyr_cache_kept's second pointer), "re-encode" when it counts
 *           from 0. head_dim at most 256.
 *   swiglu  out = silu(gate) * up, n elements.
 *   argmax  out[r] = index of the largest of x[r, 0..n), the lowest index on ties; x [rows, n].
 */
/*
 * The tensor-core linear layers wait on their copies with bounded waits; a wait that runs out is
 * recorded in a status word the library keeps per GPU (the glue calls have no cache handle).
 * pyr_glue_status synchronises `stream` and reports 0 or PYR_ERR_TIMEOUT for the current GPU since the
 * last report (reading clears the record); after a timeout the outputs of the calls since then are
 * undefined. Allocates nothing.
 */
pyr_status_t pyr_glue_status(void* stream, int32_t* host_status);
pyr_status_t pyr_glue_embed(const int32_t* ids, const void* table, void* out, int64_t tokens, int32_t d, int32_t vocab,
                            int32_t dtype, int32_t* dev_status, void* stream);
pyr_status_t pyr_glue_rmsnorm(const void* x, const void* gain, void* out, int64_t tokens, int32_t d, float eps,
                              int32_t dtype, void* stream);
pyr_status_t pyr_glue_linear(const void* x, const void* w, const void* residual, void* y, int64_t m, int32_t n,
                             int32_t k, int32_t dtype, void* stream);
pyr_status_t pyr_glue_rmsnorm_rows(const void* x, const int32_t* rows, int64_t rows_stride, const void* gain, void* out,
                                   int32_t batch, int32_t n_src, int32_t n_dst, int32_t d, float eps, int32_t dtype,
                                   void* stream);
pyr_status_t pyr_glue_linear_rows(const void* x, const void* w, const void* residual, const int32_t* res_rows,
                                  int64_t rows_stride, void* y, int32_t batch, int32_t n_src, int32_t n_dst, int32_t n,
                                  int32_t k, int32_t dtype, void* stream);
pyr_status_t pyr_glue_linear_split(const void* x, const void* w, void* const* ys, int32_t n_parts, int64_t m, int32_t part_n,
                                   int32_t k, int32_t dtype, void* stream);
pyr_status_t pyr_glue_linear_swiglu(const void* x, const void* w_gate, const void* w_up, void* out, int64_t m, int32_t n,
                                    int32_t k, int32_t dtype, void* stream);
pyr_status_t pyr_glue_rope(void* x, const int32_t* pos, int64_t tokens, int32_t n_heads, int32_t head_dim,
                           int32_t dtype, void* stream);
pyr_status_t pyr_glue_swiglu(const void* gate, const void* up, void* out, int64_t n, int32_t dtype, void* stream);
pyr_status_t pyr_glue_argmax(const void* x, int32_t* out, int64_t rows, int32_t n, int32_t dtype, void* stream);

const char* pyr_status_string(pyr_status_t status);

/* Number of kernels this process has launched through the library so far. */
uint64_t pyr_launch_count(void);

/* Library version: major*10000 + minor*100 + patch. */
int32_t pyr_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PYR_H_ */
