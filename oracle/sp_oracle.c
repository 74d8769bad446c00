/*
 * CPU oracle for the superposition-prompting hot path (arXiv 2404.06910).
 *
 * TEST INFRASTRUCTURE.  This file defines what the CUDA library must compute; it is
 * deliberately plain and slow: naive loops, explicit key sets, two-pass softmax,
 * float inputs with double arithmetic.  It shares no code, header, table or helper
 * with the CUDA path and must never be called from it.  Only the test-suite, the
 * smoke check and the CPU-baseline leg of the benchmark may load it.
 *
 * Each function cites the passage of the paper it restates.  Readings taken where
 * the paper is silent or garbled are marked "Reading:".
 *
 * Parity pins: every function below is pinned by the CPU tests against closed
 * forms, invariants, library routines or brute force, except the RoPE pairing
 * convention (half-split vs interleaved), which the paper does not fix:
 * "parity unpinned" for that one choice (both conventions are offered).
 *
 * All arrays are host memory.  Functions return 0 on success, a negative code on
 * invalid arguments.  OpenMP runs independent rows / paths in parallel only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int spo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------
 * O1  Position assignment.  Section 3.2.2, Eq. 1 (harmonic mean S(D)), Eq. 3
 * (ArangePositions a_Delta(s0, m) = <s0, s0+Delta, ..., s0+(m-1)Delta>), Algorithm 1.
 *
 *   preamble:  a_1(0, P)                       = 0, 1, ..., P-1
 *   S(D)     = N / sum_i (1 / L_i)                                     (Eq. 1)
 *   doc i:     s_i = S / L_i ;  a_{s_i}(max(preamble)+1, L_i) = P + j*s_i      (Alg. 1)
 *   query:     a_1(q0, Q) shared by every path (Algorithm 3 passes one query
 *              position array to the batched call).
 *
 * Reading (Eq. 3 prints s_1 and n for s_0 and m): the arithmetic progression above.
 * Reading (query start, Algorithm 3): the printed max(doc_1 positions) depends on which
 *   document is first and collides with that document's last token; q_mode 0 uses
 *   q0 = P + S, the next equilibrium slot, identical for every path
 *   (P + L_i * s_i = P + S for all i); q_mode 1 is the literal P + (L_1-1)*s_1.
 * Reading (zero-length documents): they hold no tokens and are left out of Eq. 1.
 * Reading (P = 0): max of an empty preamble + 1 is taken as 0.
 *
 * scheme 0 = equilibrium, 1 = left-aligned (Section 3.2.2: every doc at P + j; the
 * query starts after the longest document).
 * Output: pos[P + sum(L_i + Q)] in packed order [pre | doc_0 qry_0 | doc_1 qry_1 ...];
 * *S_out receives S(D) (equilibrium) or max L (left-aligned); *next_out receives the
 * position that follows the query (task / response tokens continue from there with
 * step 1 -- Reading: the paper never defines those positions).
 * ---------------------------------------------------------------------------------- */
int spo_positions(int scheme, int q_mode, int P, int N, const int32_t *L, int Q,
                  double *pos, double *S_out, double *next_out)
{
    if (P < 0 || N < 0 || Q < 0 || (N > 0 && !L) || !pos) return -1;
    for (int j = 0; j < P; ++j) pos[j] = (double)j;

    double S = 0.0, q0;
    if (scheme == 0) {
        double inv = 0.0;
        int n_nonempty = 0;
        for (int i = 0; i < N; ++i) {
            if (L[i] < 0) return -1;
            if (L[i] > 0) { inv += 1.0 / (double)L[i]; ++n_nonempty; }
        }
        S = n_nonempty ? (double)n_nonempty / inv : 0.0;
        q0 = (double)P + S;
        if (q_mode == 1 && N > 0 && L[0] > 0) q0 = (double)P + (double)(L[0] - 1) * (S / (double)L[0]);
    } else if (scheme == 1) {
        int mx = 0;
        for (int i = 0; i < N; ++i) { if (L[i] < 0) return -1; if (L[i] > mx) mx = L[i]; }
        S = (double)mx;
        q0 = (double)P + S;
    } else {
        return -1;
    }

    size_t r = (size_t)P;
    for (int i = 0; i < N; ++i) {
        double step = (scheme == 0) ? (L[i] > 0 ? S / (double)L[i] : 0.0) : 1.0;
        for (int j = 0; j < L[i]; ++j) pos[r++] = (double)P + (double)j * step;
        for (int j = 0; j < Q; ++j) pos[r++] = q0 + (double)j;
    }
    if (S_out) *S_out = S;
    if (next_out) *next_out = q0 + (double)Q;
    return 0;
}

/* ------------------------------------------------------------------------------------
 * O2  Rotary position encoding at real-valued positions.  Section 3.2.2, footnote on
 * RoPE: the argument of the sinusoids is interpolated linearly, i.e. evaluated at the
 * real position.  For pair m = 0..rot_dim/2-1:  theta = pos * base^(-2m/rot_dim),
 *   (a, b) -> (a cos(theta) - b sin(theta),  a sin(theta) + b cos(theta)).
 * pairing 0: (a, b) = (x[m], x[m + rot_dim/2])   ("half-split")
 * pairing 1: (a, b) = (x[2m], x[2m+1])           ("interleaved")
 * Reading: the paper does not say which pairing; that depends on the checkpoint.
 * x: [n_tokens, n_heads, head_dim] float, token stride ld_token elements, in place.
 * ---------------------------------------------------------------------------------- */
int spo_rope(float *x, const float *pos, int64_t n_tokens, int64_t ld_token, int n_heads,
             int head_dim, int rot_dim, double base, int pairing)
{
    if (!x || !pos || n_tokens < 0 || n_heads <= 0 || head_dim <= 0) return -1;
    if (rot_dim <= 0 || rot_dim > head_dim || (rot_dim & 1)) return -1;
    if (pairing != 0 && pairing != 1) return -1;
    const int half = rot_dim / 2;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int h = 0; h < n_heads; ++h) {
            float *v = x + t * ld_token + (int64_t)h * head_dim;
            for (int m = 0; m < half; ++m) {
                const double theta = (double)pos[t] * pow(base, -2.0 * (double)m / (double)rot_dim);
                const double c = cos(theta), s = sin(theta);
                const int ia = pairing ? 2 * m : m;
                const int ib = pairing ? 2 * m + 1 : m + half;
                const double a = v[ia], b = v[ib];
                v[ia] = (float)(a * c - b * s);
                v[ib] = (float)(a * s + b * c);
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Row bookkeeping for O3: which segment a packed row belongs to.
 * ---------------------------------------------------------------------------------- */
typedef struct {
    int32_t prompt;  /* owning prompt                                   */
    int32_t path;    /* owning path (global id), -1 for a preamble row  */
    int32_t off;     /* offset inside the preamble or inside doc+query  */
} row_info;

static int fill_row_info(int n_prompts, const int32_t *ppo, const int32_t *pre_start,
                         const int32_t *pre_len, const int32_t *path_start,
                         const int32_t *doc_len, const int32_t *qry_len, int64_t T,
                         row_info *info)
{
    for (int64_t r = 0; r < T; ++r) info[r].prompt = -1;
    for (int b = 0; b < n_prompts; ++b) {
        for (int j = 0; j < pre_len[b]; ++j) {
            int64_t r = (int64_t)pre_start[b] + j;
            if (r < 0 || r >= T || info[r].prompt != -1) return -2;
            info[r].prompt = b; info[r].path = -1; info[r].off = j;
        }
        for (int i = ppo[b]; i < ppo[b + 1]; ++i) {
            int n = doc_len[i] + qry_len[i];
            for (int j = 0; j < n; ++j) {
                int64_t r = (int64_t)path_start[i] + j;
                if (r < 0 || r >= T || info[r].prompt != -1) return -2;
                info[r].prompt = b; info[r].path = i; info[r].off = j;
            }
        }
    }
    return 0;
}

/* Dense softmax attention of one query vector over an explicit key list.
 * s_j = scale * <q, k_j> (+ bias_j);  m = max_j s_j;  LSE = m + ln sum_j exp(s_j - m);
 * o = sum_j exp(s_j - LSE) v_j.  Two passes, double arithmetic.  bias may be NULL.     */
static void attend_one(const float *qv, const float *const *kptr, const float *const *vptr,
                       int64_t nk, int D, double scale, const double *bias, double *s, float *o, float *lse)
{
    double m = -INFINITY;
    for (int64_t j = 0; j < nk; ++j) {
        double acc = 0.0;
        const float *kv = kptr[j];
        for (int d = 0; d < D; ++d) acc += (double)qv[d] * (double)kv[d];
        s[j] = acc * scale;
        if (bias) s[j] += bias[j];
        if (s[j] > m) m = s[j];
    }
    double denom = 0.0;
    for (int64_t j = 0; j < nk; ++j) denom += exp(s[j] - m);
    const double l = m + log(denom);
    double acc_o[512];
    for (int d = 0; d < D; ++d) acc_o[d] = 0.0;
    for (int64_t j = 0; j < nk; ++j) {
        const double p = exp(s[j] - l);
        const float *vv = vptr[j];
        for (int d = 0; d < D; ++d) acc_o[d] += p * (double)vv[d];
    }
    for (int d = 0; d < D; ++d) o[d] = (float)acc_o[d];
    if (lse) *lse = (float)l;
}

/* ------------------------------------------------------------------------------------
 * O3  Fork-join ("superposition") prefill attention.  Section 3.2: a token sequence v
 * attends to a sequence u iff the prompt DAG has a path u -> v; ForkJoin topology:
 * preamble -> N documents -> N query copies.  Within a segment attention is causal
 * (each LLM call is ordinary dense causal attention on its own tokens plus the KV
 * cache of its ancestors, Appendix B.3, operator LM).  Hence the key set A(r):
 *   preamble row j      : preamble rows 0..j
 *   doc_i row j         : all preamble rows of its prompt, doc_i rows 0..j
 *   query_i row j       : all preamble rows, all doc_i rows, query_i rows 0..j
 * (doc_i and query_i are adjacent in the packing, so the last two cases are
 *  "own rows 0..off".)
 * q: [T, H, D]; k, v: [T, Hkv, D]; head h reads KV head h / (H/Hkv).
 * out: [T, H, D]; lse: [H, T] natural log, may be NULL.
 * rows/n_rows: optional list of packed rows to compute (others untouched); NULL = all.
 * Reading: scale is passed explicitly (the paper does not restate 1/sqrt(D)).
 * ALiBi (Section 3.2.2 notes that real-valued positions are trivial for it): with pos [T] and
 * slopes [H] given, score(r, c) gets the additive bias -slopes[h] * |pos[r] - pos[c]|, the
 * linear distance penalty of ALiBi evaluated at the tokens' assigned (possibly fractional)
 * positions.  pos == NULL: no bias.
 * ---------------------------------------------------------------------------------- */
int spo_prefill_alibi(const float *q, const float *k, const float *v,
                      int n_prompts, const int32_t *ppo, const int32_t *pre_start,
                      const int32_t *pre_len, const int32_t *path_start, const int32_t *doc_len,
                      const int32_t *qry_len, int64_t T, int H, int Hkv, int D, double scale,
                      const float *pos, const float *slopes,
                      const int64_t *rows, int64_t n_rows, float *out, float *lse)
{
    if (!q || !k || !v || !out || H <= 0 || Hkv <= 0 || H % Hkv || D <= 0 || D > 512) return -1;
    if (pos && !slopes) return -1;
    row_info *info = (row_info *)malloc(sizeof(row_info) * (size_t)(T > 0 ? T : 1));
    if (!info) return -3;
    int rc = fill_row_info(n_prompts, ppo, pre_start, pre_len, path_start, doc_len, qry_len, T, info);
    if (rc) { free(info); return rc; }
    const int64_t n = rows ? n_rows : T;
    const int group = H / Hkv;
    int err = 0;
#pragma omp parallel
    {
        int64_t cap = 0;
        const float **kp = NULL, **vp = NULL;
        double *s = NULL, *bias = NULL;
#pragma omp for schedule(dynamic, 4)
        for (int64_t ii = 0; ii < n; ++ii) {
            const int64_t r = rows ? rows[ii] : ii;
            if (r < 0 || r >= T || info[r].prompt < 0) { if (rows) err = 1; continue; }
            const row_info ri = info[r];
            const int b = ri.prompt;
            const int64_t P = pre_len[b];
            const int64_t nk = (ri.path < 0) ? (ri.off + 1) : (P + ri.off + 1);
            if (nk > cap) {
                cap = nk * 2;
                kp = (const float **)realloc((void *)kp, sizeof(float *) * (size_t)cap);
                vp = (const float **)realloc((void *)vp, sizeof(float *) * (size_t)cap);
                s = (double *)realloc(s, sizeof(double) * (size_t)cap);
                bias = (double *)realloc(bias, sizeof(double) * (size_t)cap);
            }
            for (int h = 0; h < H; ++h) {
                const int hk = h / group;
                int64_t c = 0;
                if (ri.path < 0) {
                    for (int64_t j = 0; j <= ri.off; ++j, ++c) {
                        const int64_t kr = (int64_t)pre_start[b] + j;
                        kp[c] = k + (kr * Hkv + hk) * D; vp[c] = v + (kr * Hkv + hk) * D;
                    }
                } else {
                    for (int64_t j = 0; j < P; ++j, ++c) {
                        const int64_t kr = (int64_t)pre_start[b] + j;
                        kp[c] = k + (kr * Hkv + hk) * D; vp[c] = v + (kr * Hkv + hk) * D;
                    }
                    for (int64_t j = 0; j <= ri.off; ++j, ++c) {
                        const int64_t kr = (int64_t)path_start[ri.path] + j;
                        kp[c] = k + (kr * Hkv + hk) * D; vp[c] = v + (kr * Hkv + hk) * D;
                    }
                }
                if (pos) {
                    for (int64_t cc = 0; cc < c; ++cc) {
                        const int64_t kr = ((kp[cc] - k) / D - hk) / Hkv;      /* packed row of key cc */
                        bias[cc] = -(double)slopes[h] * fabs((double)pos[r] - (double)pos[kr]);
                    }
                }
                attend_one(q + (r * H + h) * D, kp, vp, c, D, scale, pos ? bias : NULL, s,
                           out + (r * H + h) * D, lse ? lse + (int64_t)h * T + r : NULL);
            }
        }
        free((void *)kp); free((void *)vp); free(s); free(bias);
    }
    free(info);
    return err ? -2 : 0;
}

int spo_prefill(const float *q, const float *k, const float *v,
                int n_prompts, const int32_t *ppo, const int32_t *pre_start,
                const int32_t *pre_len, const int32_t *path_start, const int32_t *doc_len,
                const int32_t *qry_len, int64_t T, int H, int Hkv, int D, double scale,
                const int64_t *rows, int64_t n_rows, float *out, float *lse)
{
    return spo_prefill_alibi(q, k, v, n_prompts, ppo, pre_start, pre_len, path_start, doc_len, qry_len, T, H, Hkv,
                             D, scale, NULL, NULL, rows, n_rows, out, lse);
}

/* ------------------------------------------------------------------------------------
 * O4  Bayesian path saliency.  Section 3.2.3 and Appendix B.1 (Eq. 2):
 *   log P(d_i | q_i, p) = log P(q_i | d_i, p) + log P(d_i | p) - C,
 * with each log-likelihood the (negated) shifted language-model cross-entropy summed
 * over the segment and divided by the segment length ("likelihood density per token").
 *   row_logp[t] = logits[t][y_t] - ( max_v logits[t][v] + ln sum_v exp(logits[t][v] - max) )
 *   score_i     = weight_i * sum_{t in path i, y_t != -1} row_logp[t]  +  prior_i
 * "Shifted": row t predicts the segment's token t+1; the last row has no target (-1).
 * Reading (Eq. 2's second line is garbled -- it prints a preamble term and no query
 *   term): the first line and the text fix the two terms; weight_i = 1/|q| and
 *   prior_i = the document term are caller inputs, the preamble term folds into C.
 * logits: [R, vocab] with row stride ld; row_off: [n_paths+1].
 * ---------------------------------------------------------------------------------- */
int spo_path_scores(const float *logits, int64_t ld, const int32_t *targets,
                    const int32_t *row_off, int n_paths, int vocab, const float *prior,
                    const float *weight, float *scores, float *row_logp)
{
    if (!logits || !targets || !row_off || !scores || vocab <= 0 || ld < vocab || n_paths < 0) return -1;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n_paths; ++i) {
        double sum = 0.0;
        for (int64_t t = row_off[i]; t < row_off[i + 1]; ++t) {
            const float *row = logits + t * ld;
            const int32_t y = targets[t];
            if (y == -1) { if (row_logp) row_logp[t] = 0.0f; continue; }
            if (y < 0 || y >= vocab) { err = 1; continue; }
            double m = -INFINITY;
            for (int c = 0; c < vocab; ++c) if ((double)row[c] > m) m = (double)row[c];
            double denom = 0.0;
            for (int c = 0; c < vocab; ++c) denom += exp((double)row[c] - m);
            const double lp = (double)row[y] - (m + log(denom));
            if (row_logp) row_logp[t] = (float)lp;
            sum += lp;
        }
        const double w = weight ? (double)weight[i] : 1.0;
        const double pr = prior ? (double)prior[i] : 0.0;
        scores[i] = (float)(w * sum + pr);
    }
    return err ? -2 : 0;
}

/* ------------------------------------------------------------------------------------
 * O5  Path pruning.  Section 3.2.3: greedily keep the top-k paths of the categorical
 * posterior; Appendix B.1: the constant C drops out because the scores are
 * soft-maxed over the prompt's paths.
 * Reading (Algorithm 3 prints argmin^K; the text says top-k, k = paths retained):
 *   keep the k LARGEST.
 * Reading (silent): ties -> lower path index first; NaN ranks below every number;
 *   k > N_b fills N_b entries and pads with -1; posterior treats NaN as -inf, and is 0
 *   everywhere when no score of the prompt is above -inf.
 * kept_idx: [B, k] global path ids in descending score; kept_post: [B, k] or NULL.
 * ---------------------------------------------------------------------------------- */
static int score_before(const float *s, int a, int b) /* 1 if a ranks before b */
{
    const int na = isnan(s[a]), nb = isnan(s[b]);
    if (na || nb) { if (na && nb) return a < b; return nb; }
    if (s[a] != s[b]) return s[a] > s[b];
    return a < b;
}

int spo_prune_topk(const float *scores, const int32_t *ppo, int n_prompts, int k,
                   int32_t *kept_idx, float *kept_post)
{
    if (!scores || !ppo || !kept_idx || k <= 0 || n_prompts < 0) return -1;
    for (int b = 0; b < n_prompts; ++b) {
        const int lo = ppo[b], n = ppo[b + 1] - ppo[b];
        if (n < 0) return -1;
        int *ord = (int *)malloc(sizeof(int) * (size_t)(n > 0 ? n : 1));
        for (int i = 0; i < n; ++i) ord[i] = lo + i;
        for (int i = 1; i < n; ++i) {            /* insertion sort: full, stable order */
            const int x = ord[i];
            int j = i - 1;
            while (j >= 0 && score_before(scores, x, ord[j])) { ord[j + 1] = ord[j]; --j; }
            ord[j + 1] = x;
        }
        double m = -INFINITY, denom = 0.0;
        for (int i = 0; i < n; ++i) if (!isnan(scores[lo + i]) && scores[lo + i] > m) m = scores[lo + i];
        if (m > -INFINITY)
            for (int i = 0; i < n; ++i) if (!isnan(scores[lo + i])) denom += exp((double)scores[lo + i] - m);
        for (int j = 0; j < k; ++j) {
            if (j < n) {
                kept_idx[b * k + j] = ord[j];
                if (kept_post) {
                    const float sc = scores[ord[j]];
                    kept_post[b * k + j] = (isnan(sc) || !(denom > 0.0)) ? 0.0f : (float)(exp((double)sc - m) / denom);
                }
            } else {
                kept_idx[b * k + j] = -1;
                if (kept_post) kept_post[b * k + j] = 0.0f;
            }
        }
        free(ord);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------
 * O6  Decode attention over the pruned cache.  Section 3.2.3 (pruned paths' KV is
 * discarded, the remaining caches are concatenated) and Algorithm 3: the cache the
 * response attends to is  preamble (+) for each kept path (doc (+) query) (+) task and
 * earlier response tokens.  One new token per prompt:
 *   keys = preamble_b  U  { doc_i U query_i : i kept }  U  tail_b[0 .. tail_len_b)
 * and dense softmax as in O3.  The caller appends the new token's K/V to the tail
 * before the call (Reading: the new token attends to itself, as in any causal LM).
 * q: [B, H, D]; k_cache, v_cache: [T, Hkv, D]; tail_k, tail_v: [B, tail_cap, Hkv, D];
 * kept_idx: [B, k] with -1 padding; out: [B, H, D]; lse: [B, H] or NULL.
 * ALiBi: with slopes [H] given, key c gets the bias -slopes[h] * |q_pos[b] - pos(c)|, where
 * pos(c) is cache_pos[row] for cache rows and tail_pos[b, j] for tail rows.  slopes == NULL:
 * no bias.
 * ---------------------------------------------------------------------------------- */
int spo_pruned_decode_alibi(const float *q, const float *k_cache, const float *v_cache,
                            int n_prompts, const int32_t *ppo, const int32_t *pre_start,
                            const int32_t *pre_len, const int32_t *path_start,
                            const int32_t *doc_len, const int32_t *qry_len,
                            const int32_t *kept_idx, int k, const float *tail_k, const float *tail_v,
                            const int32_t *tail_len, int tail_cap, int H, int Hkv, int D,
                            double scale, const float *q_pos, const float *cache_pos,
                            const float *tail_pos, const float *slopes, float *out, float *lse)
{
    if (!q || !k_cache || !v_cache || !out || H <= 0 || Hkv <= 0 || H % Hkv || D <= 0 || D > 512) return -1;
    if (slopes && (!q_pos || !cache_pos)) return -1;
    if (k < 0 || (k > 0 && !kept_idx)) return -1;
    const int group = H / Hkv;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (int b = 0; b < n_prompts; ++b) {
        for (int h = 0; h < H; ++h) {
            const int hk = h / group;
            int64_t nk = pre_len[b];
            for (int j = 0; j < k; ++j) {
                const int i = kept_idx[b * k + j];
                if (i == -1) continue;
                if (i < ppo[b] || i >= ppo[b + 1]) { err = 1; continue; }
                nk += doc_len[i] + qry_len[i];
            }
            const int tl = tail_len ? tail_len[b] : 0;
            if (tl < 0 || tl > tail_cap) { err = 1; continue; }
            nk += tl;
            if (nk == 0) {   /* nothing to attend to: zero output, LSE = -inf */
                for (int d = 0; d < D; ++d) out[((int64_t)b * H + h) * D + d] = 0.0f;
                if (lse) lse[b * H + h] = -INFINITY;
                continue;
            }
            const float **kp = (const float **)malloc(sizeof(float *) * (size_t)nk);
            const float **vp = (const float **)malloc(sizeof(float *) * (size_t)nk);
            double *s = (double *)malloc(sizeof(double) * (size_t)nk);
            double *bias = (double *)malloc(sizeof(double) * (size_t)nk);
            int64_t c = 0, n_cache;
            for (int j = 0; j < pre_len[b]; ++j, ++c) {
                const int64_t kr = (int64_t)pre_start[b] + j;
                kp[c] = k_cache + (kr * Hkv + hk) * D; vp[c] = v_cache + (kr * Hkv + hk) * D;
            }
            for (int jj = 0; jj < k; ++jj) {
                const int i = kept_idx[b * k + jj];
                if (i < ppo[b] || i >= ppo[b + 1]) continue;
                for (int j = 0; j < doc_len[i] + qry_len[i]; ++j, ++c) {
                    const int64_t kr = (int64_t)path_start[i] + j;
                    kp[c] = k_cache + (kr * Hkv + hk) * D; vp[c] = v_cache + (kr * Hkv + hk) * D;
                }
            }
            n_cache = c;
            for (int j = 0; j < tl; ++j, ++c) {
                const int64_t kr = (int64_t)b * tail_cap + j;
                kp[c] = tail_k + (kr * Hkv + hk) * D; vp[c] = tail_v + (kr * Hkv + hk) * D;
            }
            if (slopes) {
                for (int64_t cc = 0; cc < c; ++cc) {
                    const float *base = cc < n_cache ? k_cache : tail_k;
                    const int64_t kr = ((kp[cc] - base) / D - hk) / Hkv;
                    const double pk = cc < n_cache ? (double)cache_pos[kr] : (double)tail_pos[kr];
                    bias[cc] = -(double)slopes[h] * fabs((double)q_pos[b] - pk);
                }
            }
            attend_one(q + ((int64_t)b * H + h) * D, kp, vp, c, D, scale, slopes ? bias : NULL, s,
                       out + ((int64_t)b * H + h) * D, lse ? lse + b * H + h : NULL);
            free((void *)kp); free((void *)vp); free(s); free(bias);
        }
    }
    return err ? -2 : 0;
}

int spo_pruned_decode(const float *q, const float *k_cache, const float *v_cache,
                      int n_prompts, const int32_t *ppo, const int32_t *pre_start,
                      const int32_t *pre_len, const int32_t *path_start,
                      const int32_t *doc_len, const int32_t *qry_len,
                      const int32_t *kept_idx, int k, const float *tail_k, const float *tail_v,
                      const int32_t *tail_len, int tail_cap, int H, int Hkv, int D,
                      double scale, float *out, float *lse)
{
    return spo_pruned_decode_alibi(q, k_cache, v_cache, n_prompts, ppo, pre_start, pre_len, path_start, doc_len,
                                   qry_len, kept_idx, k, tail_k, tail_v, tail_len, tail_cap, H, Hkv, D, scale,
                                   NULL, NULL, NULL, NULL, out, lse);
}
