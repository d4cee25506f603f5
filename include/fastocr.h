/*
 * fastocr.h - C ABI of the FastOCR decode-step attention hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, for one transformer layer at a time (and, with
 * fastocr_decode_step, for a whole decode step), the attention work of the
 * paper's Algorithm 1 after warm-up:
 *   - focal layers attend the full KV cache and score every image token
 *     (Section 3.1.2, Eq. 2 first case),
 *   - the ceil(tau*N) best-scored image tokens become the focal-token set F,
 *   - all other layers attend only K = T u F, all text tokens plus F
 *     (Eq. 2 second case), the set being inherited from the nearest preceding
 *     focal layer (Cross-Layer Propagation) or from the previous decode step
 *     (Cross-Step Fixation Reuse, Section 3.2),
 * and never modifies, compacts or frees the cache (Section 2: no physical eviction).
 *
 * Conventions
 *   - "device" pointers are CUDA device memory owned by the caller and valid on
 *     the context's device; "host" pointers are ordinary host memory. The
 *     library allocates device memory only inside fastocr_create.
 *   - All tensor arguments are dense row-major with the index order written in
 *     brackets; bf16 means the 16-bit brain-float bit pattern.
 *   - Every compute call is asynchronous on `stream` (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream), performs no allocation and no
 *     host-device synchronisation, and may be captured into a CUDA graph.
 *   - Calls on one context must not overlap on the GPU (they share its
 *     workspace): issue them on one stream, or order the streams.
 *   - Return value: FASTOCR_OK or an error code; on error nothing was launched
 *     and fastocr_last_error(ctx) describes the problem. Argument checks are
 *     host-side only; the contents of device arrays (lengths, indices, page
 *     ids) cannot be validated without a synchronisation. The kernels force
 *     them into what the host did check, so that nothing outside the caller's
 *     buffers is addressed: seq_len[b] into [0, max_seq_len], the image span
 *     into the sequence, index-list entries into [0, vis_len), block-table
 *     entries into [0, num_pages) when num_pages is given. Every value that
 *     had to be changed is counted in a status word readable with
 *     fastocr_device_faults (the affected sequence's result is then
 *     meaningless; all other sequences are unaffected). Kept counts above
 *     vis_len[b] or above the index list's row length k_stride are clamped
 *     silently (documented behaviour, not a fault).
 *   - Arithmetic: bf16 inputs, fp32 accumulation; the two contractions of a block (q.K^T, P.V) run
 *     on the tensor cores (warp-level mma, bf16 x bf16 -> fp32), P split into a bf16 high part and a
 *     bf16 remainder; exponentials are ex2.approx. Outputs agree with an fp32 CPU evaluation of the
 *     same formulas to about 1e-4 absolute.
 *   - head_dim must be 128 and num_q_heads / num_kv_heads (the GQA group size)
 *     1 to 8; query head h reads KV head h / group size.
 */
#ifndef FASTOCR_H_
#define FASTOCR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum fastocr_status {
  FASTOCR_OK = 0,
  FASTOCR_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, inconsistent shapes            */
  FASTOCR_ERR_UNSUPPORTED = 2, /* head_dim != 128, group size, page size, vis_len too large   */
  FASTOCR_ERR_WORKSPACE = 3,   /* the call exceeds the limits given to fastocr_create         */
  FASTOCR_ERR_CUDA = 4         /* a CUDA runtime call failed; see fastocr_last_error          */
} fastocr_status;

typedef struct fastocr_ctx fastocr_ctx; /* opaque; owns the workspace; bound to one device */

/* Upper bounds used to size the workspace once. */
typedef struct fastocr_limits {
  int32_t max_batch;    /* sequences per call                                   */
  int32_t num_q_heads;  /* H                                                     */
  int32_t num_kv_heads; /* H_kv                                                  */
  int32_t max_seq_len;  /* cached tokens per sequence (text + image)            */
  int32_t max_vis_len;  /* image tokens per sequence, N; at most 32768          */
} fastocr_limits;

/*
 * Read-only view of ONE layer's KV cache for a (possibly ragged) batch.
 * The image tokens of sequence b occupy the contiguous position span
 * [vis_start[b], vis_start[b] + vis_len[b]); every other position is text
 * (system, prompt, generated and the current token) and is always attended.
 * One kernel launch covers up to 512 (sequence, KV head) pairs; a larger batch is processed by
 * every entry point as chunks of whole sequences, launch after launch on the stream (sequences
 * are independent of one another, so the results are those of one call; in a decode step each
 * chunk runs all its layers before the next chunk starts, and a scores_exchange callback is
 * called once per chunk and focal layer).
 */
typedef struct fastocr_kv_view {
  int32_t batch;        /* B                                                                     */
  int32_t num_q_heads;  /* H                                                                     */
  int32_t num_kv_heads; /* H_kv, divides H                                                       */
  int32_t head_dim;     /* 128                                                                   */
  int32_t page_size;    /* 0: contiguous cache; otherwise tokens per page (a power of two)       */
  int32_t max_seq_len;  /* host-known upper bound on seq_len[b]; sizes the launch                */
  const void* k;        /* device bf16. contiguous: [B][seq_stride_tokens][H_kv][128]            */
  const void* v;        /*              paged:      [num_pages][page_size][H_kv][128]            */
  int64_t seq_stride_tokens;  /* contiguous only: tokens between consecutive sequences           */
  const int32_t* block_table; /* paged only: device [B][max_pages], physical page of each logical page */
  int32_t max_pages;          /* paged only: row length of block_table                           */
  int32_t num_pages;          /* paged only: pages in the k / v pools; block-table entries outside
                                 [0, num_pages) are clamped on the device and counted as faults.
                                 0 = not given: entries are used as they are                        */
  const int32_t* seq_len;     /* device [B]: S_b, number of cached tokens                        */
  const int32_t* vis_start;   /* device [B]: first image position                                */
  const int32_t* vis_len;     /* device [B]: N_b, number of image tokens                         */
  float sm_scale;             /* softmax scale, 1/sqrt(head_dim) (Appendix B)                    */
} fastocr_kv_view;

/* Creates a context on `device` with workspace for the given limits (cudaMalloc happens here and
 * only here). *out is set on success. Not thread-safe per context. */
fastocr_status fastocr_create(fastocr_ctx** out, int device, const fastocr_limits* limits);
void fastocr_destroy(fastocr_ctx* ctx);
/* Message of the last failed call on this context (owned by the context; "" if none). */
const char* fastocr_last_error(const fastocr_ctx* ctx);
/* Synchronises the device and returns how many out-of-range indices kernels have clamped since
 * the last call (diagnostic; not for the hot path). Negative on CUDA error. */
int64_t fastocr_device_faults(fastocr_ctx* ctx);

/* |F| = ceil(tau * N) clamped to [0, N] (Section 3.1.2). tau = 0 keeps no image token,
 * tau >= 1 keeps all. Host-only. */
int32_t fastocr_kept_count(int32_t n_vis, double tau);

/*
 * Dense decode attention over the whole cache: Eq. 2 first case, Attn = softmax(q K^T * sm_scale) V
 * (Appendix B), for every query head of every sequence. This is the focal-layer path and the
 * unpruned baseline.
 *   q          device bf16 [B][H][128]
 *   out        device [B][H][128], bf16, or fp32 when out_is_fp32 != 0
 *   scores_out NULL, or device fp32 [B][n_stride]: additionally receives the head-averaged image
 *              attention of fastocr_focal_scores from the same pass over K (entries
 *              [vis_len[b], n_stride) are left untouched); n_stride >= max vis_len.
 *   image_mass_out NULL, or device fp32 [B]: Eq. 1's image-attention ratio r of this layer (the sum
 *              of those scores over the image span), from the same pass; what a warm-up step records
 *              (Section 3.1.1). May be asked for without scores_out.
 */
fastocr_status fastocr_dense_decode_attn(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, void* out,
                                         int out_is_fp32, float* scores_out, int32_t n_stride, float* image_mass_out,
                                         void* stream);

/*
 * Focal scores: for image token i of sequence b, the attention weight from the current query to
 * that token, softmax taken over the FULL cache, averaged over all H query heads (the a-bar of
 * Section 3.1.1 that Eq. 2's TopK ranks). Reads K only.
 *   scores_out     device fp32 [B][n_stride]
 *   image_mass_out NULL, or device fp32 [B]: sum_i scores = Eq. 1's image-attention ratio r
 */
fastocr_status fastocr_focal_scores(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q, float* scores_out,
                                    int32_t n_stride, float* image_mass_out, void* stream);

/*
 * TopK of Eq. 2: for each sequence the k[b] image tokens with the largest scores. Larger score
 * wins; equal scores: the lower index wins; -0 equals +0; NaN ranks below every number. Indices
 * are relative to vis_start and written in ascending order to idx_out[b][0..k[b]); the rest of the
 * row is left untouched.
 *   scores  device fp32 [B][n_stride]      vis_len device int32 [B]
 *   k       device int32 [B], 0 <= k[b] <= vis_len[b] (larger values are clamped)
 *   idx_out device int32 [B][k_stride]
 *   max_vis_len host-known bound on vis_len[b] (<= 32768)
 */
fastocr_status fastocr_select_topk(fastocr_ctx* ctx, const float* scores, int32_t n_stride, const int32_t* vis_len,
                                   const int32_t* k, int32_t batch, int32_t max_vis_len, int32_t* idx_out,
                                   int32_t k_stride, void* stream);

/*
 * Pruned decode attention: Eq. 2 second case. Softmax and weighted sum run over the kept set
 * K = T u F only: every text position plus positions vis_start + idx[b][i], i < k[b].
 *   idx device int32 [B][k_stride] (values in [0, vis_len[b]); need not be sorted, must be distinct)
 *   k   device int32 [B]
 *   max_kept host-known bound on k[b] + seq_len[b] - vis_len[b], or 0 if unknown; only used to
 *            size the launch (a long pass takes every CTA slot, a short one leaves room for the next layer)
 * A sequence whose kept set is empty yields zeros.
 */
fastocr_status fastocr_sparse_decode_attn(fastocr_ctx* ctx, const fastocr_kv_view* kv, const void* q,
                                          const int32_t* idx, const int32_t* k, int32_t k_stride, int32_t max_kept,
                                          void* out, int out_is_fp32, void* stream);

/*
 * One post-warm-up decode step of Algorithm 1 over L layers (Cross-Step Fixation Reuse followed by
 * Cross-Layer Propagation), all launches on `stream`:
 *   layer 0 reuses `fixation` when it is not focal and has_fixation != 0, otherwise it attends the
 *   full cache and selects (the fallback); each later focal layer attends the full cache and
 *   refreshes the set; every other layer attends text + the current set. On return (in stream
 *   order) `fixation` holds the set of the deepest focal layer: the F_last of the next step.
 *   layers   host array [L] of views (all with the same batch / heads / spans)
 *   q, out   device [L][B][H][128]; out bf16 or fp32; q and out must not overlap (consecutive
 *            pruned layers are launched so that one may start while the previous one drains)
 *   is_focal host uint8 [L]: membership in the focal layer set C
 *   k        device int32 [B]; fixation device int32 [B][k_stride] (in/out)
 *   max_vis_len, max_kept: host bounds as above
 * Returns through *has_fixation_out (may be NULL) whether `fixation` is valid afterwards.
 */
fastocr_status fastocr_decode_step(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers,
                                   const void* q, void* out, int out_is_fp32, const uint8_t* is_focal,
                                   const int32_t* k, int32_t* fixation, int32_t k_stride, int has_fixation,
                                   int32_t max_vis_len, int32_t max_kept, int* has_fixation_out, void* stream);

/*
 * The same step with options (NULL options = fastocr_decode_step):
 *   is_focal_seq / is_focal_seq_dev  per-sequence focal layer sets (Section 3.1.1 and Appendix E: C is
 *       profiled per sample): the matrix [L][B] of memberships, once in host memory (the library
 *       decides the launches from it) and once in device memory (the kernels read a layer's row to
 *       tell which sequences take part in a launch); both or neither. It replaces is_focal, which
 *       may then be NULL. A layer that is focal for some sequences only runs as a pruned pass over
 *       the others followed by a full pass and a selection over those. The caller uploads the device
 *       copy once, C being frozen after warm-up.
 *   union_sets  a variant, not Algorithm 1: the kept image set after a focal layer is the union of the
 *       sets selected so far in this step (Section 3.1.1 calls the union over the focal layers the
 *       aggregated focal token set); the first selection of a step replaces what was borrowed from
 *       the previous step. `fixation` still receives every focal layer's own selection, so that what
 *       is carried to the next step is the deepest focal layer's set as in Algorithm 1. The union
 *       lives in the context's workspace; max_kept must bound text + union size.
 *   scores_exchange  for a cache that is sharded by KV head over several processes (each holds
 *       num_q_heads / n query heads and their KV heads of every sequence): the focal score of
 *       Section 3.1.1 averages the attention weight over ALL heads, so the per-rank partial
 *       averages must be added up before the selection; nothing else in the step crosses ranks.
 *       When the callback is set, a focal layer runs as: full-cache pass over the local heads,
 *       local score = mean over the local heads, scores_exchange(...), selection from the exchanged
 *       scores. The callback is called on the host, between those launches, once per focal layer
 *       (the fallback at layer 0 included; per chunk of the batch, see fastocr_kv_view), in layer order; it must enqueue on `stream` an
 *       in-place sum over the ranks of scores[batch][n_stride] (device fp32, the context's
 *       workspace; entries beyond a sequence's vis_len, and rows of sequences for which the layer
 *       is not focal, hold garbage and may be summed or not) and return 0, or non-zero on failure
 *       (the step then returns FASTOCR_ERR_CUDA with nothing further launched). All ranks must run
 *       the same schedule (same focal sets, same has_fixation) and see the same k and spans; with
 *       equal head counts per rank the sum of the local means ranks the tokens as the global mean
 *       does, and every rank then selects the same set from identical scores.
 */
typedef int (*fastocr_scores_exchange_fn)(float* scores, int32_t batch, int32_t n_stride, int32_t layer,
                                          void* stream, void* user);
typedef struct fastocr_step_options {
  const uint8_t* is_focal_seq;     /* host uint8 [L][B], or NULL   */
  const uint8_t* is_focal_seq_dev; /* device uint8 [L][B], or NULL */
  int32_t union_sets;              /* 0 = Algorithm 1              */
  fastocr_scores_exchange_fn scores_exchange;   /* NULL = all heads are local */
  void* scores_exchange_user;      /* passed through to the callback */
} fastocr_step_options;
fastocr_status fastocr_decode_step_ex(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers,
                                      const void* q, void* out, int out_is_fp32, const uint8_t* is_focal,
                                      const int32_t* k, int32_t* fixation, int32_t k_stride, int has_fixation,
                                      int32_t max_vis_len, int32_t max_kept, int* has_fixation_out,
                                      const fastocr_step_options* options, void* stream);

/*
 * One warm-up step (Algorithm 1, profiling block; Section 3.1.1): nothing is pruned, every layer
 * attends the full cache, and Eq. 1's image-attention ratio is recorded for every layer and
 * sequence from the same pass over K that produces the layer's output.
 *   layers, q, out as in fastocr_decode_step
 *   ratio_out device fp32 [L][B]: r of layer l and sequence b at this step; the caller averages
 *             the w steps' records per sequence and hands the means to fastocr_focal_layers
 */
fastocr_status fastocr_warmup_step(fastocr_ctx* ctx, int32_t num_layers, const fastocr_kv_view* layers, const void* q,
                                   void* out, int out_is_fp32, float* ratio_out, void* stream);

/*
 * Focal Layer Selection (Section 3.1.1; Algorithm 1, profiling block), host-only: rank layers by
 * mean image-attention ratio (descending; equal ratios: lower layer first) and accept greedily
 * while fewer than floor(rho*L) are chosen and the candidate is more than `gap` layers from every
 * accepted one. mean_ratio host [L]; focal_out host int32 [L] receives the set in ascending order.
 * Returns the number of focal layers, or -1 on invalid arguments.
 */
int32_t fastocr_focal_layers(const double* mean_ratio, int32_t num_layers, double rho, int32_t gap,
                             int32_t* focal_out);

/* Appendix B: self-attention FLOPs of one decode step, b*l*(8h^2 + 4hs). Host-only. */
double fastocr_attn_flops(double batch, double layers, double hidden, double seq_len);
/* The same count for a pruned step, as Tables 1 and 2 print it for the method: every layer pays the
 * projections, `full_layers` of them attend seq_len tokens, the others kept_len tokens. Host-only. */
double fastocr_attn_flops_pruned(double batch, double layers, double hidden, double seq_len, double full_layers,
                                 double kept_len);

/*
 * Pruned decode attention without a context and without any allocation (the paper has no
 * counterpart; this exists for callers that cannot call cudaMalloc: engines that give all of HBM
 * to their own pool at start-up, allocator-tracked frameworks, decode loops that must stay out of
 * the driver's allocator). Same computation and arguments as fastocr_sparse_decode_attn, but the
 * scratch of the split merge is a fixed array inside the library (about 3.1 MB of device memory
 * on every GPU that loads it, held until the process exits) instead of a context's workspace.
 *   - Limit: batch * num_kv_heads <= FASTOCR_NOALLOC_MAX_UNITS, else FASTOCR_ERR_WORKSPACE.
 *   - The first call on each device resolves the array's device address and sets kernel
 *     attributes (no allocation); make that first call outside any stream capture. First calls
 *     from several host threads are serialised by the library.
 *   - All calls on a device share the one array, which keeps the previous call's contents (the
 *     entry point re-zeroes the counters it needs on `stream` before launching). Two calls that
 *     may overlap on the GPU (different streams without ordering) race on it: serialise them.
 *   - Runs on the current device; every pointer must belong to it. No cudaMalloc, cudaFree or
 *     allocating library routine is called. Errors: return code + fastocr_noalloc_last_error()
 *     (thread-local string).
 */
#define FASTOCR_NOALLOC_MAX_UNITS 256
fastocr_status fastocr_sparse_decode_attn_noalloc(const fastocr_kv_view* kv, const void* q, const int32_t* idx,
                                                  const int32_t* k, int32_t k_stride, void* out, int out_is_fp32,
                                                  void* stream);
const char* fastocr_noalloc_last_error(void);
/* Counterpart of fastocr_device_faults for the allocation-free entry point (the paper has no
 * counterpart): synchronises the current device and returns how many device-side lengths, index-list
 * or block-table entries its kernels have had to force into range on this device since the last
 * call; clears the count. Not for the hot path. Negative on CUDA error. */
int64_t fastocr_noalloc_device_faults(void);

/*
 * Optional per-kernel timing (the paper has no counterpart; measurement aid). Between
 * fastocr_profile_begin and fastocr_profile_end the launches of this context are bracketed by CUDA
 * events on their stream. With coalesce_runs == 0 every launch gets its own event pair: the figures
 * are isolated-kernel times (the event records keep consecutive layers from overlapping and the
 * interval includes launch latency). With coalesce_runs != 0 a maximal run of consecutive launches
 * of the same class shares one pair, nothing is recorded inside the run, and total time / launches
 * is the duration per launch as it occurs in an unprofiled step. fastocr_profile_begin creates
 * `max_launches` event pairs (not a hot-path call; launches beyond that are not timed);
 * fastocr_profile_end synchronises, adds up elapsed milliseconds and launch counts per kernel class
 * into the two host arrays of length FASTOCR_PROF_CLASSES, and destroys the events. Use one stream
 * between begin and end, and not while a stream is being captured.
 */
enum {
  FASTOCR_PROF_ATTN_DENSE = 0,  /* split-KV attention kernel, full cache, K and V          */
  FASTOCR_PROF_ATTN_KEYS = 1,   /* same kernel, keys only (stand-alone scoring)             */
  FASTOCR_PROF_ATTN_SPARSE = 2, /* same kernel over the kept set                            */
  FASTOCR_PROF_FINALIZE = 3,    /* logits -> head-averaged scores                           */
  FASTOCR_PROF_TOPK = 4,        /* selection                                                */
  FASTOCR_PROF_MASS = 5,        /* image-mass reduction                                     */
  FASTOCR_PROF_CLASSES = 6
};
fastocr_status fastocr_profile_begin(fastocr_ctx* ctx, int32_t max_launches, int coalesce_runs);
fastocr_status fastocr_profile_end(fastocr_ctx* ctx, double* ms_per_class, int64_t* launches_per_class);

/* Number of kernels this library has launched on any context since load (for bench accounting). */
int64_t fastocr_launch_count(void);

/* Of those, the pruned-attention launches that ran one thread-block cluster per (sequence, KV head)
 * unit, whose pieces are merged through distributed shared memory instead of global memory (chosen
 * by the library for short passes over sequences of similar length; Eq. 2 second case either way).
 * For tests and tuning. */
int64_t fastocr_cluster_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTOCR_H_ */
