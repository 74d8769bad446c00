/*
 * sp.h -- C ABI of the superposition-prompting hot path for NVIDIA B200 (sm_100a).
 *
 * Superposition prompting (arXiv 2404.06910) arranges a retrieval-augmented prompt as a
 * fork-join DAG: one shared preamble, N documents processed as parallel paths, one copy
 * of the query per path; paths are scored by the likelihood of their query copy, the
 * top-k are kept, and the response is decoded over the preamble plus the kept paths.
 * This library is the attention / scoring / pruning arithmetic of that pipeline.
 *
 * Conventions
 *  - Every function returns an sp_status; nothing throws.  sp_last_error() returns a
 *    thread-local message for the last non-zero status of the calling thread.
 *  - Unless marked HOST, every pointer is DEVICE memory owned by the caller.  The
 *    library allocates no device memory and keeps no state between calls; scratch
 *    memory is passed in as (ws, ws_bytes), sized by the *_workspace_bytes functions.
 *  - All calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL =
 *    default stream).  Arguments the host can check are checked before any launch.
 *  - Device-detected problems (a bounded wait that ran out; a layout whose device arrays
 *    contradict the host scalars: a segment outside [0, T), a length above max_pre_len /
 *    max_path_len, a negative length) are recorded in the first 4 bytes of the workspace and
 *    read back by sp_check_status().  The layout arrays live in device memory, so without a
 *    host_mirror the host cannot see them: the kernels check them instead, skip what is
 *    inconsistent (nothing outside the caller's tensors is read or written) and report it.
 *    The library built with -DSP_DEBUG_BOUNDS additionally checks every pair of segments for
 *    overlap on the device.
 *  - Tensors are dense, row-major.  Data pointers must be 16-byte aligned and
 *    n_heads * head_dim * element size must be a multiple of 16 bytes.
 *  - dtype selects storage: SP_F32 (float) or SP_BF16 (bfloat16).  Accumulation is
 *    always fp32; sp_rope_apply evaluates angles in fp64.
 *
 * Packed token layout (sp_layout).  Prompt b owns paths [prompt_path_off[b],
 * prompt_path_off[b+1]).  Its preamble occupies packed rows [pre_start[b], pre_start[b]
 * + pre_len[b]).  Path i occupies rows [path_start[i], path_start[i] + doc_len[i] +
 * qry_len[i]): the document first, its query copy right after it.  Segments must not
 * overlap.  Q is [T, n_heads, head_dim]; K, V are [T, n_kv_heads, head_dim].
 */
#ifndef SP_H_
#define SP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SP_OK = 0,
    SP_ERR_INVALID_ARG = 1,   /* a host-checkable argument is wrong; nothing was launched */
    SP_ERR_UNSUPPORTED = 2,   /* valid but not implemented (e.g. head_dim)                */
    SP_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small               */
    SP_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed                      */
    SP_ERR_TIMEOUT = 5,       /* a bounded device-side wait expired (sp_check_status)     */
    SP_ERR_LAYOUT = 6         /* the device-resident layout arrays are inconsistent
                                 (sp_check_status; the affected segments were skipped)    */
} sp_status;

enum { SP_F32 = 0, SP_BF16 = 1 };
enum { SP_ROWS_ALL = 0, SP_ROWS_QUERY_ONLY = 1 };
enum { SP_POS_EQUILIBRIUM = 0, SP_POS_LEFT_ALIGNED = 1 };
enum { SP_ROPE_HALF_SPLIT = 0, SP_ROPE_INTERLEAVED = 1 };

/* HOST copies of the six index arrays of an sp_layout (same lengths and meaning). */
typedef struct {
    const int32_t *prompt_path_off, *pre_start, *pre_len, *path_start, *doc_len, *qry_len;
} sp_layout_host;

typedef struct {
    int32_t n_prompts;               /* B                                                  */
    int32_t n_paths;                 /* NP = total paths over all prompts                  */
    const int32_t *prompt_path_off;  /* [B+1]                                              */
    const int32_t *pre_start;        /* [B]                                                */
    const int32_t *pre_len;          /* [B]                                                */
    const int32_t *path_start;       /* [NP]                                               */
    const int32_t *doc_len;          /* [NP]                                               */
    const int32_t *qry_len;          /* [NP]                                               */
    int64_t total_tokens;            /* T: number of packed rows of Q / K / V / out        */
    int32_t max_pre_len;             /* >= every pre_len[b]            (host scalar)       */
    int32_t max_path_len;            /* >= every doc_len[i]+qry_len[i] (host scalar)       */
    const sp_layout_host *host_mirror; /* HOST, nullable: when given, every call validates the
                                        whole layout on the host before launching (offsets
                                        ascending, lengths >= 0 and within the two maxima, every
                                        segment inside [0, T), no two segments overlapping) and
                                        returns SP_ERR_INVALID_ARG on a violation              */
} sp_layout;

/* Message for the calling thread's last failing call ("" if none).  HOST. */
const char *sp_last_error(void);

/* Library version string, e.g. "sp-b200 0.1".  HOST. */
const char *sp_version(void);

/*
 * Token positions of one prompt (Section 3.2.2; Eq. 1; Eq. 3; Algorithm 1).  HOST only.
 * Equilibrium: preamble 0..P-1; S = N / sum_i 1/L_i (documents of length 0 are left out);
 * document i at P + j*S/L_i; the query copy of every path at q0 + j with q0 = P + S
 * (q_mode 0) or, as Algorithm 3 prints it, the last position of document 1 (q_mode 1).
 * Left-aligned: documents at P + j, query after the longest document.
 * doc_len: HOST [n_docs].  pos: HOST [P + sum(L_i) + n_docs*Q] floats, packed order
 * [preamble | doc_0 query_0 | doc_1 query_1 | ...].  S_out / next_pos_out (nullable):
 * S(D) and the first position after the query (task and response tokens continue from
 * it with step 1).  Positions are computed in double and rounded once to float.
 */
int sp_positions(int scheme, int q_mode, int pre_len, int n_docs, const int32_t *doc_len,
                 int qry_len, float *pos, double *S_out, double *next_pos_out);

/*
 * Rotary position encoding at real-valued positions (Section 3.2.2, footnote: the
 * argument of the sinusoid is evaluated at the interpolated position).  In place.
 * x: [n_tokens, n_heads, head_dim], token stride ld_token elements (>= n_heads*head_dim).
 * pos: [n_tokens] float.  For pair m < rot_dim/2: theta = pos * base^(-2m/rot_dim),
 * (a, b) <- (a cos - b sin, a sin + b cos); pairing SP_ROPE_HALF_SPLIT pairs
 * (x[m], x[m+rot_dim/2]), SP_ROPE_INTERLEAVED pairs (x[2m], x[2m+1]).
 * rot_dim even, 2 <= rot_dim <= head_dim <= 256.  No workspace.
 */
int sp_rope_apply(void *x, const float *pos, int64_t n_tokens, int64_t ld_token, int n_heads,
                  int head_dim, int rot_dim, double base, int pairing, int dtype, void *stream);

/*
 * The same rotation for two tensors that share their positions, in one launch: a step's
 * queries xq [n_tokens, n_heads_q, head_dim] (token stride ld_q) and keys xk [n_tokens,
 * n_heads_k, head_dim] (token stride ld_k).  Each angle is evaluated once for both.
 * Equivalent to two sp_rope_apply calls; same argument rules, same dtype for both tensors.
 */
int sp_rope_apply_pair(void *xq, int64_t ld_q, int n_heads_q, void *xk, int64_t ld_k, int n_heads_k,
                       const float *pos, int64_t n_tokens, int head_dim, int rot_dim, double base,
                       int pairing, int dtype, void *stream);

/*
 * Fork-join ("superposition") prefill attention (Section 3.2: a segment attends to
 * another iff the prompt DAG has a path to it; ForkJoin topology preamble -> documents ->
 * query copies; every call is dense causal attention on its own tokens plus the KV of
 * its ancestors).  For packed row r:  out[r] = softmax(scale * q[r] K(r)^T) V(r),
 * lse[h][r] = ln sum_k exp(scale * q[r].k), where the key set K(r) is
 *   preamble row j        : preamble rows 0..j of the same prompt
 *   path i, offset j      : every preamble row of its prompt + rows 0..j of path i.
 * q: [T, n_heads, D]; k, v: [T, n_kv_heads, D] (n_heads % n_kv_heads == 0);
 * out: [T, n_heads, D]; lse: fp32 [n_heads, T] or NULL.
 * rows = SP_ROWS_ALL computes every row; SP_ROWS_QUERY_ONLY computes only the query rows
 * of every path (the cached, online case of Algorithm 3); other rows of out are untouched.
 * head_dim in {64, 128}.  SP_BF16 with head_dim 128 runs on the tensor cores (the
 * softmax probabilities are rounded to bf16 before the second product); everything else
 * runs an fp32 SIMT kernel.
 * ws: at least sp_prefill_workspace_bytes() bytes, 256-byte aligned.
 */
size_t sp_prefill_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len,
                                  int n_heads, int head_dim, int dtype);
int sp_superpose_prefill(const void *q, const void *k, const void *v, const sp_layout *lay,
                         int n_heads, int n_kv_heads, int head_dim, float scale, int rows,
                         void *out, float *lse, void *ws, size_t ws_bytes, int dtype,
                         void *stream);

/*
 * Bayesian path saliency (Section 3.2.3; Appendix B.1, Eq. 2): each path's score is the
 * length-normalised log-likelihood of its query copy plus a document prior,
 *   row_logp[t] = logits[t][y_t] - logsumexp_v logits[t][v]        (0 where y_t == -1)
 *   scores[i]   = weight[i] * sum_{t in [row_off[i], row_off[i+1])} row_logp[t] + prior[i].
 * The cross-entropy is "shifted": row t is scored against the segment's token t+1 and the
 * last row has target -1.  logits: [R, vocab], row stride ld_logits elements, rows
 * path-major, finite values; targets: int32 [R] in [-1, vocab); row_off: int32
 * [n_paths+1]; prior / weight: fp32 [n_paths] or NULL (0 / 1).  scores: fp32 [n_paths];
 * row_logp: fp32 [R] or NULL (then the workspace holds it).  n_rows = R (host scalar).
 * Targets outside [-1, vocab) score as -1.  One pass over the logits; sums run in a fixed
 * order, so results are reproducible bit for bit.
 */
size_t sp_path_scores_workspace_bytes(int64_t n_rows);
int sp_path_scores(const void *logits, int64_t ld_logits, const int32_t *targets,
                   const int32_t *row_off, int64_t n_rows, int n_paths, int vocab,
                   const float *prior, const float *weight, float *scores, float *row_logp,
                   void *ws, size_t ws_bytes, int dtype, void *stream);

/*
 * Path pruning (Section 3.2.3: greedily keep the top-k of the posterior over paths;
 * Appendix B.1: the scores are soft-maxed over the prompt's paths, so a common constant is
 * irrelevant).  Per prompt b: kept_idx[b][0..k) = global ids of the k largest scores in
 * descending order; equal scores keep the lower id first; NaN ranks below every number;
 * if the prompt has fewer than k paths the rest is -1.  kept_post (nullable): softmax of
 * the prompt's scores at the kept ids (NaN counts as -inf; 0 for padding and when no
 * score of the prompt is above -inf).  1 <= k.  No workspace.
 */
int sp_prune_topk(const float *scores, const int32_t *prompt_path_off, int n_prompts, int k,
                  int32_t *kept_idx, float *kept_post, void *stream);

/*
 * Decode attention over the pruned cache (Section 3.2.3: the KV of pruned paths is
 * dropped and the rest concatenated; Algorithm 3: the response attends to preamble +
 * kept (document + query) + task and response tokens).  One query token per prompt:
 *   keys(b) = preamble_b  U  { path i : i in kept_idx[b], i != -1 }  U  tail_b[0..tail_len[b])
 *   out[b][h] = softmax(scale * q[b][h] . K) V ;  lse[b][h] = ln sum exp(...)
 * Pruning is an index list: nothing is copied.  The caller appends the new token's K/V to
 * the tail before the call, so the token attends to itself.
 * q: [B, n_heads, D]; k_cache, v_cache: [T, n_kv_heads, D] as in the prefill;
 * kept_idx: int32 [B, k] (device; typically sp_prune_topk's output); tail_k, tail_v:
 * [B, tail_cap, n_kv_heads, D] (nullable when tail_cap == 0); tail_len: int32 [B];
 * out: [B, n_heads, D]; lse: fp32 [B, n_heads] or NULL.  head_dim in {64, 128}.
 * A prompt with no key at all gets out = 0 and lse = -inf.
 * max_keys: host upper bound on any prompt's key count (sizes the KV split);
 * pass 0 to use max_pre_len + k * max_path_len + tail_cap.
 * ws: at least sp_decode_workspace_bytes() bytes, 256-byte aligned.  The key sequence of a
 * (prompt, KV head) is split over the blocks of one thread-block cluster, which merge their
 * partial results through distributed shared memory in split order (results do not depend on
 * scheduling); the workspace is therefore not written, and its status word is not touched
 * (this call has no bounded waits).  Query heads that share a KV head (n_kv_heads < n_heads) are
 * served by one block per KV head, in groups of 4, 2 or 1, so K and V rows are read once per group.
 */
size_t sp_decode_workspace_bytes(int n_prompts, int n_heads, int head_dim);
int sp_pruned_decode(const void *q, const void *k_cache, const void *v_cache,
                     const sp_layout *lay, const int32_t *kept_idx, int k,
                     const void *tail_k, const void *tail_v, const int32_t *tail_len,
                     int tail_cap, int64_t max_keys, int n_heads, int n_kv_heads, int head_dim,
                     float scale, void *out, float *lse, void *ws, size_t ws_bytes, int dtype,
                     void *stream);

/*
 * The prefill with the rotation of Q folded in (Section 3.2.2, footnote on RoPE: the sinusoid's
 * argument is evaluated at the interpolated position).  q arrives UNROTATED and is not modified:
 * every 128-row query tile is rotated in shared memory, at the positions pos[T], between its
 * arrival and its first use, with the arithmetic of sp_rope_apply (rot_dim = head_dim), so the
 * result equals sp_rope_apply(q) followed by sp_superpose_prefill(rows = SP_ROWS_ALL) and one
 * read and one write of Q are saved.  k must already be rotated (sp_rope_apply): it is the cache
 * the decode step reads.  pos: fp32 [T] (sp_positions per prompt); base, pairing as for
 * sp_rope_apply.  bf16 with head_dim 128 only; anything else returns SP_ERR_UNSUPPORTED (rotate
 * with sp_rope_apply and call sp_superpose_prefill).  Workspace: sp_prefill_rope_workspace_bytes
 * (the tile list plus a (cos, sin) table of total_tokens x 64 pairs, 512 bytes per token); the
 * status word and sp_check_status work as for sp_superpose_prefill.
 */
size_t sp_prefill_rope_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len,
                                       int64_t total_tokens, int n_heads, int head_dim, int dtype);
int sp_superpose_prefill_rope(const void *q, const void *k, const void *v, const sp_layout *lay,
                              const float *pos, double base, int pairing, int n_heads, int n_kv_heads,
                              int head_dim, float scale, void *out, float *lse, void *ws, size_t ws_bytes,
                              int dtype, void *stream);

/*
 * ALiBi variants (Section 3.2.2: the equilibrium assignment yields real-valued positions, which
 * the ALiBi encoding takes as they are; Section 3.2.1: with ALiBi, position gaps turn into
 * attention penalties, which is what the equilibrium assignment avoids).  They compute what
 * sp_superpose_prefill / sp_pruned_decode compute with the additive bias
 *   -slopes[h] * |pos(query) - pos(key)|
 * on every admitted score before the softmax.  pos: fp32 [T], the position of every packed
 * row (sp_positions per prompt); slopes: fp32 [n_heads], >= 0.  For the decode step:
 * q_pos fp32 [B] (the new token's position), cache_pos fp32 [T] (positions of the cache
 * rows), tail_pos fp32 [B, tail_cap] (positions of the tail rows; nullable when tail_cap == 0).
 * All other arguments, workspaces, layouts and error codes are those of the plain entry
 * points; Q and K are used as given (no rotary embedding is implied).
 */
int sp_superpose_prefill_alibi(const void *q, const void *k, const void *v, const sp_layout *lay,
                               const float *pos, const float *slopes, int n_heads, int n_kv_heads,
                               int head_dim, float scale, int rows, void *out, float *lse, void *ws,
                               size_t ws_bytes, int dtype, void *stream);
int sp_pruned_decode_alibi(const void *q, const void *k_cache, const void *v_cache,
                           const sp_layout *lay, const int32_t *kept_idx, int k,
                           const void *tail_k, const void *tail_v, const int32_t *tail_len,
                           int tail_cap, int64_t max_keys, const float *q_pos, const float *cache_pos,
                           const float *tail_pos, const float *slopes, int n_heads, int n_kv_heads,
                           int head_dim, float scale, void *out, float *lse, void *ws, size_t ws_bytes,
                           int dtype, void *stream);

/*
 * Decode step with the rotary embedding folded in (Section 3.2.2 footnote: the sinusoid is
 * evaluated at the token's real-valued position).  Computes what
 *   sp_rope_apply_pair(q, newest tail key, positions q_pos)  followed by  sp_pruned_decode
 * computes, in one launch: q [B, n_heads, D] and the newest tail key row
 * tail_k[b][tail_len[b] - 1] arrive unrotated; both are rotated at position q_pos[b] (fp32 [B],
 * device; angles formed in fp64, results rounded to the storage type as the stand-alone
 * rotation does), and the rotated key row is written back in place, so later steps find it
 * rotated like every older row.  q itself is not modified.  A prompt with tail_len[b] == 0 has
 * no new key.  rope_base > 0; pairing as in sp_rope_apply; the rotation spans the whole head
 * (rot_dim == head_dim).  n_heads / n_kv_heads must be 1, 2 or 4 (one block has to own the new
 * key row); other ratios return SP_ERR_UNSUPPORTED: rotate separately and call
 * sp_pruned_decode.  No workspace; all other arguments as for sp_pruned_decode.
 */
int sp_pruned_decode_rope(const void *q, const void *k_cache, const void *v_cache,
                          const sp_layout *lay, const int32_t *kept_idx, int k, void *tail_k,
                          const void *tail_v, const int32_t *tail_len, int tail_cap, int64_t max_keys,
                          const float *q_pos, double rope_base, int pairing, int n_heads,
                          int n_kv_heads, int head_dim, float scale, void *out, float *lse, int dtype,
                          void *stream);

/*
 * Decode attention without a caller workspace.  (The paper has no counterpart: this entry
 * point exists for integration reasons only.)  It computes exactly what sp_pruned_decode
 * computes, with the same arguments minus (ws, ws_bytes), for callers that are not able to
 * obtain device memory at the point of the call: code running inside a serving engine
 * whose memory pool is fully handed out, plugins that are forbidden to call the CUDA
 * allocator, or call sites where an allocation would stall the pipeline.  The split-KV
 * scratch (arrival counters and per-split partial results) lives in one fixed
 * 8 MiB array that is part of the library image; every GPU on which the library is used
 * holds that array from load until the process exits.
 *  - Limit: n_prompts*n_heads*4 bytes of counters (rounded up to 256) plus, when the key
 *    sequence is split, n_prompts*n_heads*n_splits*(head_dim+2)*4 bytes of partials must
 *    fit in sp_pruned_decode_static_max_bytes(); otherwise SP_ERR_WORKSPACE is returned and
 *    nothing is launched (use sp_pruned_decode with your own workspace then).
 *  - The call allocates and frees nothing.  The first call on each device looks up the
 *    array's device address (a one-time runtime query made with that device current);
 *    make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the previous call
 *    left in it; each call clears the counters it needs on `stream` first.  Two calls
 *    whose kernels can overlap on the GPU (different streams, no ordering between them)
 *    race on the array: order them, or give one of them sp_pruned_decode and a workspace.
 *  - No device status word is kept for this variant.
 */
size_t sp_pruned_decode_static_max_bytes(void);
int sp_pruned_decode_static(const void *q, const void *k_cache, const void *v_cache,
                            const sp_layout *lay, const int32_t *kept_idx, int k,
                            const void *tail_k, const void *tail_v, const int32_t *tail_len,
                            int tail_cap, int64_t max_keys, int n_heads, int n_kv_heads,
                            int head_dim, float scale, void *out, float *lse, int dtype,
                            void *stream);

/*
 * Reads the device status word at the start of a workspace after synchronising `stream`.
 * Returns SP_OK, SP_ERR_TIMEOUT (a bounded wait expired; the outputs of that call are
 * not valid), SP_ERR_LAYOUT (the layout arrays on the device were inconsistent; what could not
 * be trusted was skipped, so the outputs are incomplete) or SP_ERR_CUDA.  The word is cleared
 * by the next sp_superpose_prefill / sp_pruned_decode call that uses the workspace;
 * sp_path_scores has nothing to report and leaves the word alone.
 */
int sp_check_status(const void *ws, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SP_H_ */
