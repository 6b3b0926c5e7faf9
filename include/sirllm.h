/*
 * sirllm.h - C ABI of the B200 (sm_100a) retention pass of SirLLM
 * (Yao, Li, Zhao, "SirLLM: Streaming Infinite Retentive LLM").
 *
 * One dialogue round of one or more independent streams is
 *     score  ->  append  ->  decay  ->  select  ->  compact E  ->  compact KV
 * (Algorithm 1, with the eviction of turn t+1 moved to the end of turn t).  The
 * calls below expose the three parts and the whole round.
 *
 * Conventions shared by every call
 *   - All data pointers are DEVICE pointers unless an argument is marked (host).
 *     The library allocates nothing and keeps no device state between calls; the
 *     caller owns every buffer, including the workspace `ws`
 *     (sirllm_workspace_bytes() bytes, 256-byte aligned, set up once with
 *     sirllm_workspace_init()).  On the host it remembers, per device, a few properties
 *     it would otherwise ask the runtime for at every call (SM count, shared-memory
 *     limit, the occupancy of its gather kernel).  Launches carry NVTX ranges
 *     ("sirllm:score", "sirllm:decay_select", "sirllm:compact_kv", ...).
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls validate their arguments on the host, enqueue work on that stream and
 *     return without synchronising (sirllm_status() is the exception).  Two calls
 *     that use the same workspace must be ordered on the same stream.
 *   - Return value: SIRLLM_OK or a negative SIRLLM_ERR_* code.  Every argument check
 *     runs on the host before the first copy or launch: when NULL, BAD_CONFIG, ALIGN or
 *     TOO_LARGE is returned nothing was enqueued and no buffer was touched.
 *     SIRLLM_ERR_CUDA reports a runtime call that failed, possibly part-way through the
 *     call's sequence.  Conditions only the device can see are OR-ed into a sticky
 *     status word in `ws` (SIRLLM_STATUS_* bits).
 *   - Layouts.  Logits: row-major rows of `vocab` elements, `logits_row_stride`
 *     elements apart; stream s owns rows [s*max_new, s*max_new + n_new[s]).
 *     K and V: each one contiguous array [n_streams][n_layers][n_kv_heads]
 *     [capacity][head_dim] of 16-bit elements; a "plane" is one [capacity][head_dim]
 *     slice, a "slot" one row of it.  Scores E: fp32 [n_streams][capacity].
 *     keep_idx: int32 [n_streams][threshold].  Per-stream scalars: [n_streams].
 */
#ifndef SIRLLM_H
#define SIRLLM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element types */
#define SIRLLM_F32 0
#define SIRLLM_BF16 1
#define SIRLLM_F16 2

/* return codes */
#define SIRLLM_OK 0
#define SIRLLM_ERR_NULL (-1)       /* a required pointer is NULL */
#define SIRLLM_ERR_BAD_CONFIG (-2) /* inconsistent or unsupported sirllm_config */
#define SIRLLM_ERR_ALIGN (-3)      /* a pointer or stride breaks the 16-byte alignment rule */
#define SIRLLM_ERR_CUDA (-4)       /* a CUDA runtime call failed; see sirllm_last_cuda_error() */
#define SIRLLM_ERR_TOO_LARGE (-5)  /* the problem exceeds a fixed limit of the entry point */

/* bits of the device status word */
#define SIRLLM_STATUS_TOKEN_RANGE 1 /* a token id outside [0, vocab) other than -1; scored 0 */
#define SIRLLM_STATUS_OVERFLOW 2    /* live_len + n_new > capacity; that stream's round was skipped */
#define SIRLLM_STATUS_TIMEOUT 4     /* a bounded device-side wait gave up; results are unreliable */
#define SIRLLM_STATUS_BAD_KEEP 8    /* a caller-supplied keep list is not strictly ascending within
                                       [0, capacity); that stream was not compacted */

/* comparison policies of Section 4.1.1 for sirllm_keep_policy */
#define SIRLLM_POLICY_STREAM 1
#define SIRLLM_POLICY_RANDOM 2
#define SIRLLM_POLICY_INTERVAL 3

/* pairing of a key row's elements under rotary embedding, for sirllm_rerotate_keys */
#define SIRLLM_ROPE_HALF 0        /* pair i = (row[i], row[i + head_dim/2]) */
#define SIRLLM_ROPE_INTERLEAVED 1 /* pair i = (row[2i], row[2i+1]) */

/* Largest `capacity` the selection kernel supports (the scores of one stream are
 * held in one SM's shared memory). */
#define SIRLLM_MAX_CAPACITY 49152
/* Largest `head_dim` (K/V rows of at most 1 KB; the gather stages 32 rows per copy). */
#define SIRLLM_MAX_HEAD_DIM 512

typedef struct sirllm_config {
    int32_t n_streams;   /* independent dialogue streams, >= 1 */
    int32_t n_layers;    /* K/V planes per stream = n_layers * n_kv_heads (each of K and V) */
    int32_t n_kv_heads;
    int32_t head_dim;    /* elements per K/V row, a multiple of 8, <= SIRLLM_MAX_HEAD_DIM */
    int32_t capacity;    /* physical slots per plane, <= SIRLLM_MAX_CAPACITY */
    int32_t budget;      /* retained slots after an eviction = n_sink + n_recent + k  (the
                            "cache size" of Tables 1-3) */
    int32_t n_sink;      /* attention-sink slots always kept: the first n_sink (Section 3.1) */
    int32_t n_recent;    /* most recent slots always kept (Section 3.1; 0 in the SirLLM rows) */
    int32_t threshold;   /* evict only when live_len > threshold (the L of Algorithm 1);
                            budget <= threshold <= capacity */
    int32_t max_new;     /* most tokens one stream appends per round; logits rows per stream */
    int32_t kv_dtype;    /* SIRLLM_BF16 or SIRLLM_F16 (rows are only copied) */
    int32_t logits_dtype;/* SIRLLM_F32 or SIRLLM_BF16 */
    int64_t vocab;       /* V */
    int64_t logits_row_stride; /* elements between consecutive logits rows, >= vocab */
} sirllm_config;

/* Bytes of device workspace the calls below need for this configuration (0 if the
 * configuration is invalid).  Host-only, pure.  No counterpart in the paper. */
size_t sirllm_workspace_bytes(const sirllm_config *cfg);

/* Zeroes the workspace (status word, scratch).  Call once after allocating it.
 * No counterpart in the paper. */
int sirllm_workspace_init(const sirllm_config *cfg, void *ws, void *cuda_stream);

/*
 * Token Entropy (Section 3.2, the equation defining e_i = -log P(x_i | x_0..x_{i-1}),
 * natural logarithm): for every stream s and t < n_new[s],
 *     out_entropy[s*max_new + t] = -log softmax(logits row)[token_ids[s*max_new + t]]
 * computed as one streaming log-sum-exp over the vocabulary in fp32 (final
 * combination in fp64).  Row t must be the distribution token t was drawn from; the
 * library does no shifting.  token id -1 = "no prediction for this position" -> 0.
 * Any other id outside [0, vocab) -> 0 and SIRLLM_STATUS_TOKEN_RANGE.
 *   logits      [n_streams*max_new rows] fp32 or bf16, read once, never written
 *   token_ids   int32 [n_streams*max_new]
 *   n_new       int32 [n_streams], or NULL meaning max_new for every stream
 *   out_entropy fp32 [n_streams*max_new]; entries t >= n_new[s] are left untouched
 * Logits must be finite or -inf, with at least one finite entry per row.
 */
int sirllm_score(const sirllm_config *cfg, const void *logits, const int32_t *token_ids,
                 const int32_t *n_new, float *out_entropy, void *ws, void *cuda_stream);

/*
 * Token Entropy without re-reading the logits (Section 3.2: the same e_i, and its remark
 * that the score is obtained while the token is generated, at no extra cost).  A producer -
 * an LM-head GEMM whose epilogue reduces each output tile as it is computed - hands over,
 * for every logits row, n_tiles pairs and the target logit instead of the row itself:
 *     pairs[row][i] = (m_i, s_i),  m_i = max of tile i's logits,  s_i = sum_tile exp(z - m_i)
 *     target_logit[row] = z[row][token_ids[row]]
 * and  e = log(sum_i s_i * exp(m_i)) - target_logit  (natural log, fp64 combine).  A tile
 * with s_i = 0 (fully masked) is ignored.  Token ids are only checked (-1 -> 0, out of
 * range -> 0 and SIRLLM_STATUS_TOKEN_RANGE).  Row and stream layout as in sirllm_score.
 *   pairs            float[2] x [n_streams*max_new][pair_row_stride], 8-byte aligned
 *   n_tiles          pairs used per row (>= 1);  pair_row_stride >= n_tiles, in pairs
 *   target_logit     fp32 [n_streams*max_new]
 */
int sirllm_score_pairs(const sirllm_config *cfg, const void *pairs, int32_t n_tiles,
                       int64_t pair_row_stride, const float *target_logit,
                       const int32_t *token_ids, const int32_t *n_new, float *out_entropy,
                       void *ws, void *cuda_stream);

/*
 * Token Entropy under a vocabulary-parallel LM head (Section 3.2: the same e_i; the sum over
 * the vocabulary inside its softmax splits over column ranges).  The caller holds columns
 * [col0, col0 + n_cols) of every logits row - one rank's shard - and gets, per row,
 *     pairs_out[row * pair_stride] = (m, s) with  sum over the range of exp(z) = s * exp(m),
 *                                    m within rounding of the range's largest logit
 *                                    ((0, 0) for an empty or fully masked range)
 *     target_out[row] = z[row][token_ids[row]] if that column lies in the range, else 0
 * Ranks exchange these few bytes per row (all-gather of the pairs, sum of the targets) and
 * finish with sirllm_score_pairs, n_tiles = number of ranks; cfg->vocab stays the FULL
 * vocabulary (token ids are checked against it there).  Rows and streams as in sirllm_score.
 *   logits_slice      [n_streams*max_new rows] of n_cols elements, slice_row_stride apart
 *                     (may be NULL when n_cols is 0: a rank that owns no column)
 *   pairs_out         float[2] x [rows * pair_stride], 8-byte aligned; pair_stride >= 1 lets a
 *                     rank write straight into its column of a [rows][ranks] array
 *   target_out        fp32 [rows]
 * Rows at or beyond n_new[s] are left untouched.
 */
int sirllm_score_partial(const sirllm_config *cfg, const void *logits_slice, int64_t col0,
                         int64_t n_cols, int64_t slice_row_stride, const int32_t *token_ids,
                         const int32_t *n_new, void *pairs_out, int64_t pair_stride,
                         float *target_out, void *ws, void *cuda_stream);

/*
 * sirllm_score for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a packaging variant of the same kernel.)
 *
 * Who needs it: code that runs where every device allocation belongs to someone else - a
 * plugin or custom-op slot inside a host framework that passes fixed inputs and outputs and
 * no scratch - or that must not call the allocator at that moment because an allocation
 * can synchronise the whole device or fail when memory is tight.  Such a caller has no
 * place to put the workspace sirllm_score wants, so this entry point takes none: its
 * scratch (the per-row tickets and per-CTA partial sums, 590080 bytes) is a fixed array
 * inside the library image.  It calls no cudaMalloc / cudaFree and no allocating routine.
 *
 * Same arguments and result as sirllm_score (scores are bit-identical), except:
 *   status   int32 device word that receives SIRLLM_STATUS_* bits (OR-ed in; the caller
 *            zeroes it), or NULL to drop them
 *   limits   n_streams * max_new <= 16384 rows, and rows * ceil(vocab / 32768 [bf16] or
 *            16384 [fp32]) <= 65536; beyond that SIRLLM_ERR_TOO_LARGE is returned and
 *            nothing runs
 * Things to know:
 *   - every GPU that loads the library holds the array until the process exits;
 *   - the first call on each device looks up the array's address on that device (the
 *     device must be current, as for any call here); make that first call before any
 *     stream capture starts;
 *   - all calls on a device share the array: each call clears the part that must start
 *     at zero with a memset on `cuda_stream`, so calls ordered on one stream are safe, but
 *     two calls that can overlap on the GPU (different streams, no dependency) race.
 */
int sirllm_score_static(const sirllm_config *cfg, const void *logits, const int32_t *token_ids,
                        const int32_t *n_new, float *out_entropy, int32_t *status,
                        void *cuda_stream);

/*
 * Memory decay and selection (Section 3.3: E = E x eta_decay, Id_entropy = Top_k(E);
 * Section 3.1: Id_sink, Id_recent; Algorithm 1's test "KV cache size > L").
 * For every stream: scores[s][i] <- fp32(scores[s][i] * decay[s]) for i < live_len[s]
 * (one IEEE multiply, denormals kept); then if live_len[s] <= threshold the keep list
 * is the identity 0..live_len-1, else it is, in ascending order,
 *     [0, n_sink)  U  top-k of [n_sink, live_len - n_recent)  U  [live_len - n_recent, live_len)
 * with k = budget - n_sink - n_recent.  Ranking: higher score first by the total
 * order on fp32 bit patterns (negatives below positives, -0 < +0); equal scores ->
 * the lower slot wins.  Exactly one keep list is correct.
 *   scores   fp32 [n_streams][capacity], updated in place
 *   serial   int64 [n_streams][capacity] or NULL: an 8-byte tag per slot (e.g. the
 *            token's text position) that travels with the scores when they are compacted
 *   live_len int32 [n_streams]; rewritten to n_keep only if compact_scores != 0
 *   decay    fp32 [n_streams]
 *   keep_idx int32 [n_streams][threshold] out;  n_keep int32 [n_streams] out
 *   compact_scores != 0: also scores[s][j] <- scores[s][keep[j]] (and serial), j < n_keep
 */
int sirllm_decay_select(const sirllm_config *cfg, float *scores, int64_t *serial, int32_t *live_len,
                        const float *decay, int32_t *keep_idx, int32_t *n_keep,
                        int32_t compact_scores, void *ws, void *cuda_stream);

/*
 * Keep lists of the paper's comparison policies (Section 4.1.1), in the format of
 * sirllm_decay_select so that they feed sirllm_compact_kv unchanged.  Nothing is evicted
 * while live_len[s] <= threshold (identity list); otherwise, in ascending order,
 *   SIRLLM_POLICY_STREAM    sinks and the most recent budget - n_sink slots (StreamLLM)
 *   SIRLLM_POLICY_INTERVAL  sinks, then every interval-th slot behind them, interval =
 *                           floor(live_len / budget), until k = budget - n_sink - n_recent
 *                           are taken, then the recent window (IntervalLLM)
 *   SIRLLM_POLICY_RANDOM    sinks, a uniformly random k-subset of the middle, the recent
 *                           window (RandomLLM).  Middle slot i draws the 24-bit number
 *                           philox4x32_10(counter = (i, round, stream_base + s, 0),
 *                           key = seed)[0] >> 8; the k largest stay, equal draws -> lower slot.
 * Scores, tags and live_len are not touched: these policies do not use them; the caller
 * sets live_len[s] = n_keep[s] after compacting.
 */
int sirllm_keep_policy(const sirllm_config *cfg, int32_t policy, const int32_t *live_len,
                       uint64_t seed, int32_t round, int32_t stream_base, int32_t *keep_idx,
                       int32_t *n_keep, void *ws, void *cuda_stream);

/*
 * KV gather (Section 3.1, X[Id]; Section 3.3, KV_cache = KV_cache[Id_sink, Id_entropy]):
 * for every plane p of stream s and j < n_keep[s]:  dst[p][j][:] <- src[p][keep_idx[s][j]][:].
 * Rows keep their relative order, so slot order = order in the text (the positions
 * example of Section 3.3).  k_dst == k_src (and v_dst == v_src) compacts in place;
 * otherwise source and destination must not overlap.  Either of K or V may be NULL
 * (both src and dst) to skip it.  Every keep list must be strictly ascending within
 * [0, capacity) (else SIRLLM_STATUS_BAD_KEEP and the stream is left alone).
 *
 * What the gather needs from the device, and what a time-out leaves behind.  The kernel is a
 * persistent grid (one CTA per SM, sized from the occupancy the runtime reports) whose workers
 * draw units of work from a counter in `ws`; a plane may be cut into segments that different
 * workers move, and a segment waits - a bounded number of polls - until the earlier segments of
 * its plane have read the rows it is about to overwrite.  A worker only waits for units drawn
 * before its own, by workers that are running, so the waits end however few CTAs the device
 * keeps resident (a shared or partitioned GPU makes the call slower, not wrong).  If a wait
 * does run out (a hung device, a workspace shared by two calls that overlap),
 * SIRLLM_STATUS_TIMEOUT is raised, the worker stops storing and the kernel ends: an in-place
 * cache is then PARTLY compacted - rows already stored are final, the others still hold what
 * they held before - and the caller must treat the stream's cache as lost.  The same holds for
 * sirllm_step and sirllm_step_pairs.
 */
int sirllm_compact_kv(const sirllm_config *cfg, const void *k_src, const void *v_src, void *k_dst,
                      void *v_dst, const int32_t *keep_idx, const int32_t *n_keep, void *ws,
                      void *cuda_stream);

/*
 * Positions inside the cache for models that store keys AFTER rotary position embedding
 * (Section 3.3: positions are assigned by place in the cache, not in the text; the printed
 * example gives tokens [0,1,2,3,5,7,11,12] the positions [0..7]).  Call after K has been
 * compacted with the same keep lists: the key now in slot j was written for position
 * keep_idx[s][j]; it is turned by (j - keep_idx[s][j]) positions, pair i of the row by the
 * angle shift * rope_base^(-2i/head_dim), so that it becomes the key of a token at position
 * j.  Rows that did not move are not touched.  Angles and the rotation are evaluated in fp64
 * and each element is rounded once, from fp64, to the K dtype.  (A model that caches keys before
 * the rotary embedding needs no such call: slot order already is the position.)
 *   k         the K cache of sirllm_compact_kv, updated in place; head_dim % 16 == 0
 *   rope_base the base of the frequencies (10000, 500000, ...); layout: SIRLLM_ROPE_*
 */
int sirllm_rerotate_keys(const sirllm_config *cfg, void *k, const int32_t *keep_idx,
                         const int32_t *n_keep, double rope_base, int32_t layout,
                         void *cuda_stream);

/*
 * One whole round (Algorithm 1's loop body): score the n_new[s] new tokens, append
 * their scores at scores[s][live_len[s] ...] (their K/V rows and serial tags must
 * already sit in slots [live_len[s], live_len[s] + n_new[s]) of every plane), decay
 * all scores once, and if the new length exceeds `threshold` select, compact the
 * scores (and tags) and compact K and V in place.  live_len[s] becomes the new
 * length.  If live_len[s] + n_new[s] > capacity the stream is skipped untouched and
 * SIRLLM_STATUS_OVERFLOW is raised.
 *   keep_idx, n_keep  out as in sirllm_decay_select
 *   new_entropy       fp32 [n_streams*max_new] out or NULL: the raw (undecayed) scores
 */
int sirllm_step(const sirllm_config *cfg, const void *logits, const int32_t *token_ids,
                const int32_t *n_new, float *scores, int64_t *serial, int32_t *live_len,
                const float *decay, void *k, void *v, int32_t *keep_idx, int32_t *n_keep,
                float *new_entropy, void *ws, void *cuda_stream);

/* sirllm_step whose scores come from a producer's per-tile pairs (see sirllm_score_pairs)
 * instead of the logits; everything else as in sirllm_step (Algorithm 1's loop body). */
int sirllm_step_pairs(const sirllm_config *cfg, const void *pairs, int32_t n_tiles,
                      int64_t pair_row_stride, const float *target_logit, const int32_t *token_ids,
                      const int32_t *n_new, float *scores, int64_t *serial, int32_t *live_len,
                      const float *decay, void *k, void *v, int32_t *keep_idx, int32_t *n_keep,
                      float *new_entropy, void *ws, void *cuda_stream);

/* sirllm_step with four caller-created cudaEvent_t handles (host array phase_events[4])
 * recorded on the stream before scoring, before selection, before KV compaction and
 * after it, so that a profiler-free caller can time the three phases.  The work done is
 * identical to sirllm_step.  No counterpart in the paper. */
int sirllm_step_phases(const sirllm_config *cfg, const void *logits, const int32_t *token_ids,
                       const int32_t *n_new, float *scores, int64_t *serial, int32_t *live_len,
                       const float *decay, void *k, void *v, int32_t *keep_idx, int32_t *n_keep,
                       float *new_entropy, void *ws, void *cuda_stream, void **phase_events);

/*
 * One whole round for a caller whose model outputs live in HOST memory (Algorithm 1's
 * loop body, as sirllm_step): copies the round's inputs to the device, runs
 * sirllm_step on them and copies the round's results back, all enqueued on the stream;
 * the host outputs are valid once the stream has been synchronised.  Pinned host
 * buffers let the copies run asynchronously.
 *   (host) h_logits, h_token_ids  laid out as the device arrays of sirllm_step
 *   (host) h_n_new  int32 [n_streams];  h_live_len int32 [n_streams]: the caller's copy
 *          of the current live lengths (it tells where the new K/V rows go)
 *   (host) h_new_k, h_new_v  [n_streams][planes][max_new][head_dim] the round's new rows,
 *          or NULL when the rows are already in the device caches
 *   d_logits, d_token_ids, d_n_new  device staging with the shapes sirllm_step expects
 *   scores ... new_entropy          device state and outputs exactly as in sirllm_step,
 *                                   keep_idx / n_keep / new_entropy required
 *   (host) h_keep_idx [n_streams][threshold], h_n_keep [n_streams],
 *          h_new_entropy [n_streams*max_new]  results (h_n_keep = the new live lengths)
 */
int sirllm_step_host(const sirllm_config *cfg, const void *h_logits, const int32_t *h_token_ids,
                     const int32_t *h_n_new, const void *h_new_k, const void *h_new_v,
                     const int32_t *h_live_len, void *d_logits, int32_t *d_token_ids,
                     int32_t *d_n_new, float *scores, int64_t *serial, int32_t *live_len,
                     const float *decay, void *k, void *v, int32_t *keep_idx, int32_t *n_keep,
                     float *new_entropy, int32_t *h_keep_idx, int32_t *h_n_keep,
                     float *h_new_entropy, void *ws, void *cuda_stream);

/* Exercises the failure path of the library's device-side waits without a failure: one
 * thread polls a progress word of `ws` that nothing ever sets, `polls` times (<= 2^20, a few
 * hundred milliseconds at most), gives up exactly as the KV gather would and raises
 * SIRLLM_STATUS_TIMEOUT; the GPU and the context stay usable.  Read the result with
 * sirllm_status().  No counterpart in the paper. */
int sirllm_selftest_bounded_wait(const sirllm_config *cfg, void *ws, uint32_t polls,
                                 void *cuda_stream);

/* Waits for the stream, copies the status word to *status_out (host) and, if
 * `clear` != 0, resets it.  No counterpart in the paper. */
int sirllm_status(void *ws, void *cuda_stream, int32_t *status_out, int32_t clear);

/* Text for a return code; the message of the last failed CUDA call of this thread.
 * No counterpart in the paper. */
const char *sirllm_strerror(int code);
const char *sirllm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SIRLLM_H */
