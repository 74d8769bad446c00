// Host-side pieces of the C ABI that launch nothing: error strings, layout checks,
// token position assignment, the device status read-back.
#include <cstring>
#include <utility>
#include <vector>

#include "common.cuh"

namespace sp {

char *error_buffer()
{
    static thread_local char buf[512] = {0};
    return buf;
}

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(error_buffer(), 512, fmt, ap);
    va_end(ap);
    return code;
}

// Multiprocessor count of the current device, queried once per device; grids and split counts
// are sized from it.  Without a usable device (host-only callers of the workspace sizers) the
// count of the part this library is written for is assumed.
int num_sms()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); n = 148; }
        cached[dev] = n;
    }
    return cached[dev];
}

int check_layout(const sp_layout *lay)
{
    SP_REQUIRE(lay != nullptr, SP_ERR_INVALID_ARG, "layout is NULL");
    SP_REQUIRE(lay->n_prompts >= 0 && lay->n_paths >= 0, SP_ERR_INVALID_ARG,
               "layout: negative n_prompts (%d) or n_paths (%d)", lay->n_prompts, lay->n_paths);
    SP_REQUIRE(lay->total_tokens >= 0 && lay->total_tokens < (int64_t)INT32_MAX, SP_ERR_INVALID_ARG,
               "layout: total_tokens %lld out of range", (long long)lay->total_tokens);
    SP_REQUIRE(lay->max_pre_len >= 0 && lay->max_path_len >= 0, SP_ERR_INVALID_ARG,
               "layout: negative max_pre_len / max_path_len");
    if (lay->n_prompts > 0)
        SP_REQUIRE(lay->prompt_path_off && lay->pre_start && lay->pre_len, SP_ERR_INVALID_ARG,
                   "layout: per-prompt arrays are NULL");
    if (lay->n_paths > 0)
        SP_REQUIRE(lay->path_start && lay->doc_len && lay->qry_len, SP_ERR_INVALID_ARG,
                   "layout: per-path arrays are NULL");
    if (lay->host_mirror == nullptr) return SP_OK;

    // full validation on the caller's host copy of the arrays
    const sp_layout_host &m = *lay->host_mirror;
    const int B = lay->n_prompts, NP = lay->n_paths;
    const int64_t T = lay->total_tokens;
    if (B > 0) SP_REQUIRE(m.prompt_path_off && m.pre_start && m.pre_len, SP_ERR_INVALID_ARG, "layout: host mirror of the per-prompt arrays is NULL");
    if (NP > 0) SP_REQUIRE(m.path_start && m.doc_len && m.qry_len, SP_ERR_INVALID_ARG, "layout: host mirror of the per-path arrays is NULL");
    if (B > 0) SP_REQUIRE(m.prompt_path_off[0] == 0 && m.prompt_path_off[B] == NP, SP_ERR_INVALID_ARG,
                          "layout: prompt_path_off must run from 0 to n_paths");
    std::vector<std::pair<int64_t, int64_t>> seg;          // (first row, one past the last row)
    seg.reserve((size_t)B + NP);
    for (int b = 0; b < B; ++b) {
        SP_REQUIRE(m.prompt_path_off[b] <= m.prompt_path_off[b + 1], SP_ERR_INVALID_ARG, "layout: prompt_path_off decreases at prompt %d", b);
        SP_REQUIRE(m.pre_len[b] >= 0 && m.pre_len[b] <= lay->max_pre_len, SP_ERR_INVALID_ARG,
                   "layout: pre_len[%d] = %d outside [0, max_pre_len = %d]", b, m.pre_len[b], lay->max_pre_len);
        SP_REQUIRE(m.pre_start[b] >= 0 && (int64_t)m.pre_start[b] + m.pre_len[b] <= T, SP_ERR_INVALID_ARG,
                   "layout: preamble of prompt %d leaves [0, total_tokens)", b);
        if (m.pre_len[b]) seg.emplace_back(m.pre_start[b], (int64_t)m.pre_start[b] + m.pre_len[b]);
    }
    for (int i = 0; i < NP; ++i) {
        SP_REQUIRE(m.doc_len[i] >= 0 && m.qry_len[i] >= 0 && (int64_t)m.doc_len[i] + m.qry_len[i] <= lay->max_path_len,
                   SP_ERR_INVALID_ARG, "layout: path %d has lengths (%d, %d) outside [0, max_path_len = %d]", i, m.doc_len[i],
                   m.qry_len[i], lay->max_path_len);
        const int64_t n = (int64_t)m.doc_len[i] + m.qry_len[i];
        SP_REQUIRE(m.path_start[i] >= 0 && m.path_start[i] + n <= T, SP_ERR_INVALID_ARG,
                   "layout: path %d leaves [0, total_tokens)", i);
        if (n) seg.emplace_back(m.path_start[i], m.path_start[i] + n);
    }
    std::sort(seg.begin(), seg.end());
    for (size_t i = 1; i < seg.size(); ++i)
        SP_REQUIRE(seg[i].first >= seg[i - 1].second, SP_ERR_INVALID_ARG,
                   "layout: the segments starting at rows %lld and %lld overlap", (long long)seg[i - 1].first, (long long)seg[i].first);
    return SP_OK;
}

}  // namespace sp

extern "C" {

const char *sp_last_error(void) { return sp::error_buffer(); }

const char *sp_version(void) { return "sp-b200 0.1"; }

// Section 3.2.2, Eq. 1, Eq. 3, Algorithm 1 (see sp.h).
int sp_positions(int scheme, int q_mode, int pre_len, int n_docs, const int32_t *doc_len,
                 int qry_len, float *pos, double *S_out, double *next_pos_out)
{
    SP_REQUIRE(scheme == SP_POS_EQUILIBRIUM || scheme == SP_POS_LEFT_ALIGNED, SP_ERR_INVALID_ARG,
               "sp_positions: unknown scheme %d", scheme);
    SP_REQUIRE(q_mode == 0 || q_mode == 1, SP_ERR_INVALID_ARG, "sp_positions: q_mode must be 0 or 1");
    SP_REQUIRE(pre_len >= 0 && n_docs >= 0 && qry_len >= 0, SP_ERR_INVALID_ARG,
               "sp_positions: negative length");
    SP_REQUIRE(pos != nullptr && (n_docs == 0 || doc_len != nullptr), SP_ERR_INVALID_ARG,
               "sp_positions: NULL array");
    for (int i = 0; i < n_docs; ++i)
        SP_REQUIRE(doc_len[i] >= 0, SP_ERR_INVALID_ARG, "sp_positions: doc_len[%d] < 0", i);

    const double P = (double)pre_len;
    double spacing = 0.0;   // S(D) for equilibrium, longest document for left alignment
    if (scheme == SP_POS_EQUILIBRIUM) {
        double recip = 0.0;
        int counted = 0;
        for (int i = 0; i < n_docs; ++i)
            if (doc_len[i] > 0) { recip += 1.0 / doc_len[i]; ++counted; }
        spacing = counted ? counted / recip : 0.0;
    } else {
        for (int i = 0; i < n_docs; ++i) spacing = std::fmax(spacing, (double)doc_len[i]);
    }
    double qry_first = P + spacing;
    if (scheme == SP_POS_EQUILIBRIUM && q_mode == 1 && n_docs > 0 && doc_len[0] > 0)
        qry_first = P + (doc_len[0] - 1) * (spacing / doc_len[0]);

    float *w = pos;
    for (int j = 0; j < pre_len; ++j) *w++ = (float)j;
    for (int i = 0; i < n_docs; ++i) {
        const double delta =
            scheme == SP_POS_EQUILIBRIUM ? (doc_len[i] > 0 ? spacing / doc_len[i] : 0.0) : 1.0;
        for (int j = 0; j < doc_len[i]; ++j) *w++ = (float)(P + j * delta);
        for (int j = 0; j < qry_len; ++j) *w++ = (float)(qry_first + j);
    }
    if (S_out) *S_out = spacing;
    if (next_pos_out) *next_pos_out = qry_first + qry_len;
    return SP_OK;
}

int sp_check_status(const void *ws, void *stream)
{
    SP_REQUIRE(ws != nullptr, SP_ERR_INVALID_ARG, "sp_check_status: workspace is NULL");
    uint32_t word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SP_CUDA(cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st));
    SP_CUDA(cudaStreamSynchronize(st));
    if (word == sp::STATUS_OK) return SP_OK;
    if (word == sp::STATUS_TIMEOUT)
        return sp::fail(SP_ERR_TIMEOUT, "a bounded device-side wait expired; outputs are not valid");
    if (word == sp::STATUS_BAD_LAYOUT)
        return sp::fail(SP_ERR_LAYOUT, "the layout arrays on the device are inconsistent with total_tokens / max_pre_len / "
                                       "max_path_len (or overlap); the affected segments were skipped");
    return sp::fail(SP_ERR_CUDA, "unknown device status word %u", word);
}

}  // extern "C"
