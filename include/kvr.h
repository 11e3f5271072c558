/*
 * kvr.h -- C ABI of libkvr: the data-parallel hot path of KVReviver (reversible KV-cache
 * compression with sketch-based token reconstruction) for NVIDIA B200 (sm_100a).
 *
 * Two operations, applied independently to every head-instance (batch x layer x kv head; in the
 * paper every attention layer runs its own copy of the method: Algorithm section, Overview):
 *
 *   compress          score the N context tokens by accumulated attention of an observation
 *                     window, keep the top-budget tokens exactly (Recent + Candidate parts of
 *                     Algorithm 3, one-shot form) and add every other token's key / value vector
 *                     into the r x b Vague sketch (Algorithm 1).
 *   decode attention  per decode step, rebuild every compressed token as the element-wise median
 *                     of its r sketch cells (Algorithm 2), take exact rows for the others
 *                     (Algorithm 4) and run one ordinary softmax attention,
 *                     Softmax(q K^T / sqrt(d_k)) V, over all N tokens (Overview, Calculation
 *                     Phase).  The rebuilt cache is never written to memory.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, contiguous, 16-byte aligned,
 *     unless the function name ends in _host (then it is a host pointer, pinned or pageable).
 *   - `hash_seeds` is host memory, copied during kvr_sketch_create.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     enqueue work on that stream and return without synchronising, except the _host variants and
 *     kvr_sketch_create / kvr_sketch_destroy, which synchronise.  kvr_compress runs part of its work
 *     on a stream owned by the handle, forked from and joined back into `cuda_stream` with events, so
 *     the ordering a caller sees on `cuda_stream` is unchanged.
 *   - A kvr_decode_attention call that directly follows another one of the same handle on the same
 *     stream may start while the earlier one is still finishing (programmatic dependent launch): it
 *     uses that time to stage handle-owned data that no decode call writes.  It reads q, Kr, Vr and
 *     writes `out` only after all work enqueued before it on the stream has completed, so the
 *     ordering a caller sees is unchanged.
 *   - The handle owns the sketch cells, hash tables, per-token lists, scores and workspaces.
 *     Workspaces grow on demand: the first call of a given size may call cudaMalloc.
 *   - Argument errors are reported by the return value before anything is launched; nothing
 *     throws or aborts across this boundary.  A handle is not thread-safe, and two calls that
 *     touch the same layer must be ordered on one stream.
 *   - `layer` selects the slice of the handle; KVR_ALL_LAYERS (-1) processes every layer in one
 *     launch, and every tensor then carries a leading [n_layers] axis.
 */
#ifndef KVR_H
#define KVR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KVR_OK = 0,
    KVR_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, value out of range */
    KVR_ERR_UNSUPPORTED = 2, /* legal in the paper, not built here (r = 7, head_dim != 128, ...)   */
    KVR_ERR_SHAPE = 3,       /* sizes inconsistent with the handle (N > max_context, layer, ...) */
    KVR_ERR_ALLOC = 4,       /* device allocation failed */
    KVR_ERR_CUDA = 5,        /* a CUDA runtime call or launch failed */
    KVR_ERR_STATE = 6,       /* decode / inspection of a layer that was never compressed */
    KVR_ERR_LIMIT = 7        /* the call needs more than a fixed built-in capacity */
} kvr_status_t;

typedef enum { KVR_F16 = 0, KVR_BF16 = 1 } kvr_dtype_t;

#define KVR_ALL_LAYERS (-1)
#define KVR_MAX_B 8192 /* cells per row */

/* Shape of the Vague sketch and of the model slice it serves (Vague Sketch section: r rows of
 * b cells, each cell a key vector and a value vector of head_dim elements, all zero initially). */
typedef struct {
    int32_t r;           /* rows ("buckets" in the paper): 3 (the paper's fixed value; the fast
                            kernels), or 1 / 5 (a general kernel; compress, decode and the
                            inspection calls only)                                               */
    int32_t b;           /* cells per row, 1 .. KVR_MAX_B                                        */
    int32_t head_dim;    /* d_k; only 128                                                        */
    int32_t n_kv_heads;  /* H                                                                    */
    int32_t n_q_heads;   /* Hq, a multiple of H; query head hq reads kv head hq / (Hq/H); Hq/H<=8 */
    int32_t batch;       /* B                                                                    */
    int32_t n_layers;    /* L                                                                    */
    int32_t max_context; /* largest N accepted by kvr_compress                                   */
    int32_t kv_dtype;    /* kvr_dtype_t of K, V, Qobs, q                                         */
    int32_t index_mix;   /* 1: token indices are scrambled by a fixed 32-bit bijection before
                            hashing (default); 0: raw indices (test mode: seeds A=1,C=0 give
                            h(J) = J mod b, injective once b >= N)                               */
    int32_t seeds_per_head; /* 0: one set of hash seeds for all head-instances; 1: one set per kv
                            head (hash_seeds is then [n_kv_heads][r][4]): tokens collide in
                            different cells in different heads                                  */
} kvr_sketch_desc_t;

typedef struct kvr_sketch kvr_sketch_t; /* opaque; library-owned host + device memory */

/* Create the sketch storage for batch x n_layers x n_kv_heads head-instances, zero it, and build
 * the hash tables.  The paper leaves h_i and g_i open ("r distinct hash functions" of the token
 * index J, coefficients of +-1; Vague Sketch section, Algorithms 1-2); this library uses
 *     h_i(J) = ((A_i m(J) + C_i) mod p) mod b,   g_i(J) = +1 / -1 for (A'_i m(J) + C'_i) mod p
 *     even / odd,   p = 2^31 - 1,
 * with hash_seeds[i] = {A_i, C_i, A'_i, C'_i} (host, r x 4 uint32, each < p) shared by all
 * head-instances, or one such set per kv head (desc->seeds_per_head = 1: n_kv_heads x r x 4; the
 * head-instances of a kv head share its set across batch and layers), and m the index scrambler
 * selected by desc->index_mix.
 * Errors: INVALID_ARG (NULL, seed >= p, sizes < 1), UNSUPPORTED, ALLOC, CUDA.  *out is NULL on error. */
kvr_status_t kvr_sketch_create(kvr_sketch_t** out, const kvr_sketch_desc_t* desc,
                               const uint32_t* hash_seeds, void* cuda_stream);

/* Zero the cells of one layer (or all) and forget its compressed state. */
kvr_status_t kvr_sketch_reset(kvr_sketch_t* sk, int32_t layer, void* cuda_stream);

/* Synchronise the device and free everything the handle owns.  NULL is accepted. */
kvr_status_t kvr_sketch_destroy(kvr_sketch_t* sk);

/* Device bytes currently owned by the handle (cells, tables, lists, workspaces). */
size_t kvr_sketch_device_bytes(const kvr_sketch_t* sk);

/* Compress (Algorithm 3, one-shot form; Algorithm 1 for the evicted tokens).
 *   K, V   [batch, n_kv_heads, N, head_dim]      kv_dtype
 *   Qobs   [batch, n_q_heads,  W, head_dim]      kv_dtype; the W observation queries are taken to
 *          sit after all N tokens (no mask).  score[j] = sum over the Hq/H query heads of the kv
 *          head and over the W queries of Softmax_j(q . k_j / sqrt(head_dim))  (Overview: tokens
 *          are ranked by accumulated attention scores, "the result of Softmax(QK^T)").
 *   budget R = min(budget, N) tokens are kept exactly: the newest n_recent (Recent part) plus the
 *          R - n_recent highest scores among the others (Candidate part; ties: lower index wins).
 *   Outputs, caller-allocated: Kr, Vr [batch, n_kv_heads, R, head_dim] (kv_dtype) and
 *          ret_idx [batch, n_kv_heads, R] (int32, ascending).  May be NULL when R == 0.
 * The layer's cells are zeroed first, so a layer may be compressed again.  Integer results
 * (selection given the scores, bucket and sign of every token) are exact; cells are fp32 sums
 * taken in a fixed order (ascending token index within two interleaved halves of a cell's tokens,
 * short runs added plainly and the run sums accumulated with compensation): bit-reproducible.
 * Errors: INVALID_ARG, SHAPE (N > max_context, bad layer, n_recent > R, W < 1), ALLOC, CUDA. */
kvr_status_t kvr_compress(kvr_sketch_t* sk, int32_t layer, const void* K, const void* V,
                          const void* Qobs, int32_t N, int32_t W, int32_t budget, int32_t n_recent,
                          void* Kr, void* Vr, int32_t* ret_idx, void* cuda_stream);

/* One decode step (Algorithm 4 fused with the attention of the Calculation Phase).
 *   q      [batch, n_q_heads, head_dim]  kv_dtype
 *   Kr, Vr, ret_idx: as produced by kvr_compress for this layer (the rows may be permuted
 *          together; ret_idx itself is not read by the kernels -- membership is kept in the handle)
 *   n_retained = rows of Kr / Vr per head-instance: at least the R of the layer's last kvr_compress.
 *          Rows beyond R are tokens that arrived after the compress and are kept exactly (Algorithm 3
 *          pushes a new token to the Recent part; the Overview inserts the generated token after the
 *          attention step): the caller appends their K / V rows to Kr / Vr, and the softmax then runs
 *          over the N compressed-context tokens plus those rows.
 *   softmax_scale: 0 selects 1/sqrt(head_dim).
 *   out    [batch, n_q_heads, head_dim]  float32:  Softmax over all N tokens of the layer, exact
 *          rows for retained tokens, element-wise median of three cells (values multiplied by
 *          g_i(J)) for compressed ones.
 * Errors: INVALID_ARG, SHAPE, STATE (layer not compressed), ALLOC, CUDA. */
kvr_status_t kvr_decode_attention(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr,
                                  const void* Vr, const int32_t* ret_idx, int32_t n_retained,
                                  float softmax_scale, float* out, void* cuda_stream);

/* Several queries per head over the same storage (speculative decoding, chunked prefill): the cache
 * is rebuilt once per tile of tokens (Algorithm 4, Algorithm 2 for the vague tokens) and serves all
 * queries, so the reconstruction cost of the Calculation Phase is shared (paper, Throughput Analysis:
 * the rebuild comes first, the attention after it).
 *   q    device [batch, n_q_heads, n_queries, head_dim] (kv_dtype)
 *   out  device [batch, n_q_heads, n_queries, head_dim] float32
 *   Kr, Vr, ret_idx, n_retained as in kvr_decode_attention (rows appended after the compress included).
 *   causal = 1: the last n_queries rows of the storage are the queries' own tokens, in order; query t
 *               sees the cache up to and including its own token (rows < n_retained - n_queries + t + 1).
 *   causal = 0: every query sees the whole storage.
 * The two contractions run on the tensor cores on 16-bit halves of the reconstructed vectors
 * (x = hi + lo, 22 significant bits; fp32 accumulation): reconstructed values beyond the 16-bit float
 * range (65504) are not supported.  Needs a handle with a class grid (as the staged decode kernel:
 * at most 4 query heads per kv head, b up to about 540): KVR_ERR_UNSUPPORTED otherwise.
 * Errors: INVALID_ARG, SHAPE, STATE, UNSUPPORTED, ALLOC, CUDA. */
kvr_status_t kvr_decode_attention_mq(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr,
                                     const void* Vr, const int32_t* ret_idx, int32_t n_retained,
                                     int32_t n_queries, int32_t causal, float softmax_scale, float* out,
                                     void* cuda_stream);

/* kvr_decode_attention without any allocation (the paper has no counterpart: this is a property
 * of the library, not of the method).  For callers that cannot allocate device memory when they
 * decode -- a serving process whose own pool already holds all free device memory, so that a
 * cudaMalloc would fail or eat the pool's head-room, or a decode loop that must avoid the
 * device-wide synchronisation cudaMalloc / cudaFree imply.  kvr_decode_attention may grow its
 * workspace on the first call of a given size; this form never calls cudaMalloc, cudaFree or any
 * allocating routine.  Its scratch (split partials and arrival tickets) is one fixed array of
 * KVR_STATIC_SCRATCH_BYTES in device global memory that belongs to the library image: every GPU
 * that loads libkvr holds it until the process exits.
 *   - Arguments, results and errors as kvr_decode_attention (rows appended after the compress
 *     included; the split kernel serves the call); in addition KVR_ERR_LIMIT when the
 *     call covers more than 4096 head-instances or needs more split-partial space than the array
 *     has (head-instances x splits x (n_q_heads / n_kv_heads) x 520 bytes; one layer of 8 kv
 *     heads at 32k context needs about 0.9 MiB, 256 head-instances in one launch about 1 MiB).
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current; host threads that make their first calls together are serialised by a
 *     lock); make that first call before any stream capture begins.
 *   - All calls on a device share the array, which keeps the previous call's contents; the tickets
 *     are cleared on `cuda_stream` before each launch.  Two calls whose kernels can overlap on the
 *     GPU (different streams, or different handles on different streams) race on it: keep every
 *     use of this entry point on one stream per device, or order them with events. */
#define KVR_STATIC_SCRATCH_BYTES (4u << 20)
kvr_status_t kvr_decode_attention_static(kvr_sketch_t* sk, int32_t layer, const void* q,
                                         const void* Kr, const void* Vr, const int32_t* ret_idx,
                                         int32_t n_retained, float softmax_scale, float* out,
                                         void* cuda_stream);

/* ---- generation after the compress (Algorithm 3 applied to an existing storage) ----
 *
 * While tokens are generated the caller appends their exact K / V rows to Kr / Vr (see
 * kvr_decode_attention).  The paper ranks the exactly stored tokens by accumulated attention scores
 * ("the result of Softmax(QK^T)", Overview) and, when the exact storage overflows, hands the losers
 * to the Vague sketch (kvr_accumulate_scores, kvr_demote).  The swap loop of Algorithm 3 brings a vague
 * token back when its score overtakes a candidate's: the scores of vague tokens are kept in the handle's
 * per-token array (kvr_get_scores; written by kvr_compress for every token, by kvr_demote and kvr_swap
 * for the tokens they hand to the sketch, raised by kvr_accumulate_vague_scores), the loop is kvr_swap. */

/* score_acc[row] += sum over the query heads of the kv head of the softmax probability that row
 * received in the layer's LAST kvr_decode_attention call; pass the same q, Kr, n_rows and
 * softmax_scale as in that call.  score_acc: [batch, n_kv_heads, n_rows] float32, in/out.
 * Errors: INVALID_ARG, SHAPE, STATE, CUDA. */
kvr_status_t kvr_accumulate_scores(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr,
                                   int32_t n_rows, float softmax_scale, float* score_acc,
                                   void* cuda_stream);

/* kvr_decode_attention, kvr_accumulate_scores and kvr_accumulate_vague_scores as one call: the paper's
 * Calculation Phase keeps the attention scores of the step it has just computed (Overview), it does not
 * compute them twice.  Arguments as kvr_decode_attention plus score_acc [batch, n_kv_heads, n_retained]
 * float32, in/out (as in kvr_accumulate_scores).  Where the staged decode kernel serves the call it writes
 * every logit it computes to a workspace of the handle ((n_retained + compressed tokens) x query heads per
 * kv head x 4 bytes per head-instance, allocated on first use) and one small kernel turns them into mass:
 * the cache is read once.  Where the split kernel serves it, the two accumulate kernels run after it.
 * Both give the same sums up to the order of fp32 additions inside a logit.
 * Errors: as kvr_decode_attention, ALLOC, UNSUPPORTED for r != 3. */
kvr_status_t kvr_decode_attention_scored(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr,
                                         const void* Vr, const int32_t* ret_idx, int32_t n_retained,
                                         float softmax_scale, float* out, float* score_acc, void* cuda_stream);

/* Overflow step.  Kr, Vr [batch, n_kv_heads, n_rows, head_dim] and ret_idx [.., n_rows] (ascending
 * token indices: the retained tokens of the compress followed by the appended ones) hold more than
 * `budget` rows.  Per head-instance the newest n_recent rows stay (Recent part), the budget - n_recent
 * highest row_scores among the others stay (Candidate part; equal scores: the older token stays), and
 * every other row is added to the sketch (Algorithm 1).  new_context (<= max_context) = the layer's
 * context length from now on: the old one plus the appended rows, whose token indices continue the
 * old context without gaps (n_rows - retained count = new_context - old context).
 * Outputs (caller-allocated, distinct from the inputs): Kr_out, Vr_out [.., budget, head_dim],
 * ret_idx_out [.., budget], row_scores_out [.., budget] (may be NULL).  After the call the layer
 * decodes with n_retained >= budget.
 * Errors: INVALID_ARG, SHAPE (n_rows < retained count, budget > n_rows, n_recent > budget,
 * new_context out of range), STATE, ALLOC, CUDA. */
kvr_status_t kvr_demote(kvr_sketch_t* sk, int32_t layer, const void* Kr, const void* Vr,
                        const int32_t* ret_idx, const float* row_scores, int32_t n_rows,
                        int32_t new_context, int32_t budget, int32_t n_recent, void* Kr_out, void* Vr_out,
                        int32_t* ret_idx_out, float* row_scores_out, void* cuda_stream);

/* scores[token] += attention mass (as in kvr_accumulate_scores) of every token that is held by the
 * Vague sketch, in the handle's per-token score array, under the softmax of the layer's LAST
 * kvr_decode_attention call (pass the same q and softmax_scale).  The key of a vague token is the
 * one Algorithm 2 returns.  Errors: INVALID_ARG, SHAPE, STATE, CUDA. */
kvr_status_t kvr_accumulate_vague_scores(kvr_sketch_t* sk, int32_t layer, const void* q,
                                         float softmax_scale, void* cuda_stream);

/* Swap loop of Algorithm 3, in place on the caller's exact storage of the layer.  As long as the
 * best-scored token of the Vague part beats the worst-scored Candidate row by more than the factor
 * replace_rate (and fewer than max_swaps swaps were made), the two change places: the vague token is
 * queried from the sketch and taken out of it again, the candidate's vectors go into the sketch, and
 * the queried vectors take the candidate's row.
 * Kr, Vr [batch, n_kv_heads, n_rows, head_dim] (kv_dtype), ret_idx and row_scores [.., n_rows]: the
 * storage as the layer's last kvr_compress / kvr_demote left it (n_rows = its retained count).  The
 * Candidate part is the rows [0, n_rows - n_recent); the newest n_recent rows are never touched.  A
 * swapped row receives the queried vectors rounded to kv_dtype, the vague token's index and score; the
 * candidate's vectors go into the sketch, its score into the handle's per-token array.  V.Delete is
 * Algorithm 1 with the negated vectors.  The comparison is taken in fp32; among equal scores the lower
 * token index is taken.  After swaps ret_idx is no longer ascending inside the Candidate part.
 * n_swapped: device [batch, n_kv_heads] int32, swaps made per head-instance; may be NULL.
 * The paper's ReplaceRate is 1.1.  Errors: INVALID_ARG, SHAPE (n_rows differs from the layer's retained
 * count, n_recent > n_rows), STATE, CUDA. */
kvr_status_t kvr_swap(kvr_sketch_t* sk, int32_t layer, void* Kr, void* Vr, int32_t* ret_idx,
                      float* row_scores, int32_t n_rows, int32_t n_recent, float replace_rate,
                      int32_t max_swaps, int32_t* n_swapped, void* cuda_stream);

/* Which kernel serves kvr_decode_attention (and its _host form).  Both compute the same thing:
 *   KVR_DECODE_SPLIT   one CTA per token slice, cells read from global memory through L1/L2.
 *                      Serves every configuration the library accepts.
 *   KVR_DECODE_STAGED  the compressed tokens are grouped into C x C classes by (row-1 cell mod C,
 *                      row-2 cell mod C); a CTA stages the rows-1-and-2 cells of one class in shared
 *                      memory (all 128 channels, keys and values) and walks the class in row-0-cell
 *                      order, so two of the three cells of a token come from shared memory and the
 *                      third stays in registers for a run of tokens.  Needs n_q_heads / n_kv_heads
 *                      in {1, 2, 4} and b <= about 600; when it cannot run the call uses
 *                      KVR_DECODE_SPLIT.
 *   KVR_DECODE_AUTO    (default) staged whenever it is available, unless there are so few
 *                      compressed tokens that hardly any two of a class share a row-0 cell.
 * kvr_last_decode_kernel reports which of the two the last decode call of the handle launched. */
typedef enum { KVR_DECODE_AUTO = 0, KVR_DECODE_SPLIT = 1, KVR_DECODE_STAGED = 2 } kvr_decode_kernel_t;
kvr_status_t kvr_sketch_set_decode_kernel(kvr_sketch_t* sk, int32_t which);
int32_t kvr_last_decode_kernel(const kvr_sketch_t* sk);

/* Choice of the importance-scoring kernels of kvr_compress (the paper scores tokens by "the result of
 * Softmax(QK^T)", Overview; it names no kernel).  Both produce the same scores up to the order of
 * fp32 additions.
 *   KVR_SCORE_MMA_SYNC  warp-level mma.sync tiles, keys staged with cp.async.
 *   KVR_SCORE_TCGEN05   tcgen05.mma with the accumulator in tensor memory, operands placed by TMA.
 *                       Needs at least 128 key rows and 128 observation rows in the call and 16-byte
 *                       aligned K and Qobs; where that does not hold kvr_compress returns
 *                       KVR_ERR_UNSUPPORTED when this kernel was requested explicitly.
 *   KVR_SCORE_AUTO      (default) tcgen05 whenever it is available.
 * A bounded wait of the tcgen05 kernel that gives up sets bit 1 of the device status word
 * (kvr_sketch_device_status).  kvr_last_score_kernel reports what the last compress launched. */
typedef enum { KVR_SCORE_AUTO = 0, KVR_SCORE_MMA_SYNC = 1, KVR_SCORE_TCGEN05 = 2 } kvr_score_kernel_t;

/* What the query makes of the three numbers it collects per element (Algorithm 2: "Median(res, dim=0)").
 *   KVR_COMBINE_MEDIAN (default)  their middle, as the paper prints it.
 *   KVR_COMBINE_MEAN              their mean, the other classical Count-Sketch estimator (not the
 *                                 paper's choice: a collision in one row moves the mean, not the median).
 * Applies to every call that reconstructs: kvr_decode_attention (both kernels, and the _host and
 * _static forms), kvr_reconstruct, kvr_accumulate_vague_scores, kvr_swap.  The sketch contents do not
 * depend on it, so it may be switched between calls. */
typedef enum { KVR_COMBINE_MEDIAN = 0, KVR_COMBINE_MEAN = 1 } kvr_combine_t;
kvr_status_t kvr_sketch_set_combine(kvr_sketch_t* sk, int32_t which);

/* The storage split the paper's hyper-parameter study settles on (Recent 0.45 / Candidate 0.45 / Vague
 * 0.10 of the budget, r = 3, one sketch cell counted like one token), for a context of `context`
 * tokens at compression ratio `ratio` (0 < ratio <= 1):
 *     total = floor(ratio * context + 0.5) slots;  b = max(1, floor(0.1 * total / 3 + 0.5)) cells per row;
 *     exact rows = max(0, total - 3 b), of which n_recent = exact / 2 (rounded down) are the Recent part.
 * Pass `exact_rows` as kvr_compress's budget, `n_recent` as its n_recent, `b` to kvr_sketch_create.
 * Host arithmetic only.  Errors: INVALID_ARG. */
kvr_status_t kvr_paper_storage_split(int32_t context, float ratio, int32_t* exact_rows, int32_t* n_recent, int32_t* b);

/* Per-layer budgets from per-layer weights (the paper's appendix on Fisher information: a layer's weight
 * is the summed Fisher information of its key and value projection matrices, and "is used to determine
 * the memory budget allocation ratio across different layers"; it gives no formula).  Reading taken:
 * budgets proportional to the weights, the mean budget being floor(ratio * context + 0.5) rows; a
 * layer's budget never exceeds `context` (the excess is re-shared among the other layers in
 * proportion); fractions are settled by largest remainder (ties: lower layer), so the budgets add up
 * to n_layers * mean exactly (or to n_layers * context when that is smaller).
 * weights: host [n_layers], non-negative, not all zero (computed by the caller: the library never
 * sees model weights); budgets: host [n_layers], out.  Pass budgets[l] to kvr_compress of layer l.
 * Host arithmetic only.  Errors: INVALID_ARG. */
kvr_status_t kvr_layer_budgets(const double* weights, int32_t n_layers, int32_t context, float ratio,
                               int32_t* budgets);

/* Where the observation queries of kvr_compress sit (the paper does not say).
 *   on = 0 (default)  after the context: every query sees all N keys.
 *   on = 1            the W queries of a head are the last W context tokens themselves: query t
 *                     (t = 0..W-1) is token N - W + t and sees the keys j <= N - W + t only (the
 *                     model's causal mask); its softmax runs over those keys.  Needs W <= N
 *                     (kvr_compress returns KVR_ERR_SHAPE otherwise). */
kvr_status_t kvr_sketch_set_obs_window_causal(kvr_sketch_t* sk, int32_t on);
kvr_status_t kvr_sketch_set_score_kernel(kvr_sketch_t* sk, int32_t which);
int32_t kvr_last_score_kernel(const kvr_sketch_t* sk);

/* The staged kernel receives its shared-memory copies through a hardware barrier it waits on.  The
 * wait is bounded: a CTA that has waited 0.2 s gives up, finishes with whatever it has and sets bit 0
 * of a status word in device memory instead of hanging the GPU.  This call synchronises
 * `cuda_stream` and copies the word to *status (host memory): 0 means every decode launched on this
 * handle so far completed normally; anything else means outputs since then are invalid. */
kvr_status_t kvr_sketch_device_status(kvr_sketch_t* sk, int32_t* status, void* cuda_stream);

/* Test hook for the give-up paths (no counterpart in the paper).  wait_limit_ns replaces the 0.2 s limit
 * (100 us .. 1 s); unannounced_bytes > 0 (a multiple of 16, at most 4096) makes a kernel expect that many
 * bytes more on a staging barrier than its copies deliver, so the barrier never completes:
 *   - staged decode kernel: every class CTA waits wait_limit_ns on its cells barrier, sets bit 0 of the
 *     status word and carries on with the cells, which landed long before (the outputs are still right);
 *   - tcgen05 scoring kernel: the wait for the query tile runs out, the CTA sets bit 1, skips its tiles
 *     and runs to its end, where it releases its tensor memory (the scores of that compress are void).
 * Nothing faults or hangs, and no copy is in flight when a CTA exits (the limit cannot be set below the
 * time a copy takes).  0 bytes and 200 000 000 ns restore normal operation.  Errors: INVALID_ARG. */
kvr_status_t kvr_sketch_set_wait_test(kvr_sketch_t* sk, int64_t wait_limit_ns, int32_t unannounced_bytes);

/* Algorithm 3 ("insert newly generated token(s) T and compress") as one call.  The caller's exact
 * storage of the layer holds n_rows rows per head-instance, the Candidate part first, the newest
 * n_recent rows being the Recent part.  In the algorithm's order:
 *   1. the n_new new tokens (K_new, V_new [batch, n_kv_heads, n_new, head_dim], kv_dtype) join the
 *      Recent part; their token indices continue the context, their scores start at 0;
 *   2. when the Recent part then holds more than r_budget + slack tokens, its oldest tokens, all that
 *      exceed r_budget, move to the Candidate part at once;
 *   3. while the Candidate part holds more than c_budget rows its lowest-scored row goes into the
 *      sketch (Algorithm 1; among equal scores the older token stays), its score into the handle's
 *      per-token array;
 *   4. the swap loop (as kvr_swap, with replace_rate and max_swaps).
 * How many rows remain depends on the counts only: kvr_append_sizes returns the rows (and through
 * n_recent_after the Recent rows) the storage holds afterwards, -1 for impossible counts; the caller
 * sizes Kr_out, Vr_out [batch, n_kv_heads, rows_after, head_dim], ret_idx_out and row_scores_out
 * [.., rows_after] with it (they must not alias the inputs).  Nothing is waited for between the
 * steps: every launch is enqueued on `cuda_stream`, the swap loop decides on the device.
 * n_swapped: device [batch, n_kv_heads] int32 or NULL.  After the call the handle describes the new
 * storage: pass rows_after to kvr_decode_attention.  Errors: INVALID_ARG, SHAPE (n_rows below the
 * layer's retained count, context beyond max_context), STATE, ALLOC, CUDA. */
int32_t kvr_append_sizes(int32_t n_rows, int32_t n_recent, int32_t n_new, int32_t r_budget, int32_t c_budget,
                         int32_t slack, int32_t* n_recent_after);
kvr_status_t kvr_append(kvr_sketch_t* sk, int32_t layer, const void* Kr, const void* Vr,
                        const int32_t* ret_idx, const float* row_scores, int32_t n_rows, int32_t n_recent,
                        const void* K_new, const void* V_new, int32_t n_new, int32_t r_budget,
                        int32_t c_budget, int32_t slack, float replace_rate, int32_t max_swaps,
                        void* Kr_out, void* Vr_out, int32_t* ret_idx_out, float* row_scores_out,
                        int32_t* n_swapped, void* cuda_stream);

/* Host-buffer forms of the two calls: inputs are copied host -> device inside the call, the
 * retained rows stay in a handle-owned device store (so Kr / Vr / ret_idx are not passed), and
 * the decode output is copied back to `out` before the call returns (it synchronises the stream).
 * The handle's staging buffers are allocated on first use. */
kvr_status_t kvr_compress_host(kvr_sketch_t* sk, int32_t layer, const void* K, const void* V,
                               const void* Qobs, int32_t N, int32_t W, int32_t budget,
                               int32_t n_recent, void* cuda_stream);
kvr_status_t kvr_decode_attention_host(kvr_sketch_t* sk, int32_t layer, const void* q,
                                       float softmax_scale, float* out, void* cuda_stream);

/* ---- inspection (not on the timed path); all outputs are device pointers ------------------- */

/* Importance scores of the last compress: s [batch, n_kv_heads, N] float32. */
kvr_status_t kvr_get_scores(const kvr_sketch_t* sk, int32_t layer, float* s, void* cuda_stream);

/* Compressed tokens (ascending) and their cells / coefficients:
 * cmp_idx [batch, n_kv_heads, a], bucket [batch, n_kv_heads, r, a] (int32),
 * sign [batch, n_kv_heads, r, a] (int8, +1 / -1), a = N - R.  Any pointer may be NULL. */
kvr_status_t kvr_get_assignment(const kvr_sketch_t* sk, int32_t layer, int32_t* cmp_idx,
                                int32_t* bucket, int8_t* sign, void* cuda_stream);

/* Sketch cells: [batch, n_kv_heads, 2, r, b, head_dim] float32; index 0 of the axis of size 2 is
 * the key vectors, 1 the value vectors (this is also the layout in device memory). */
kvr_status_t kvr_get_cells(const kvr_sketch_t* sk, int32_t layer, float* cells, void* cuda_stream);

/* Algorithm 2 for every compressed token, ascending: Kt, Vt [batch, n_kv_heads, a, head_dim] f32. */
kvr_status_t kvr_reconstruct(const kvr_sketch_t* sk, int32_t layer, float* Kt, float* Vt,
                             void* cuda_stream);

/* N and R recorded by the last compress of a layer (host ints); STATE if never compressed. */
kvr_status_t kvr_layer_shape(const kvr_sketch_t* sk, int32_t layer, int32_t* N, int32_t* R);

/* Calibration, not part of the method: measures on the current device the two on-chip rates that
 * bound Algorithm 2's reconstruction (the Vague Sketch section's element-wise median of r cells) --
 * fp32 min/max operations per second (peaks[0], lane operations: one min or max of one element) with a
 * register-only loop, and shared-memory bytes read per second (peaks[1]) with conflict-free 16-byte
 * loads.  peaks: host [2], out.  Synchronous: launches two short kernels on `cuda_stream`, waits for
 * them and returns; allocates and frees 512 bytes of device memory.  Errors: INVALID_ARG, ALLOC, CUDA. */
kvr_status_t kvr_measure_pipe_peaks(double* peaks, void* cuda_stream);

/* Number of kernels this library has launched on behalf of the handle since creation. */
int64_t kvr_launch_count(const kvr_sketch_t* sk);

const char* kvr_status_string(kvr_status_t st);

#ifdef __cplusplus
}
#endif
#endif /* KVR_H */
