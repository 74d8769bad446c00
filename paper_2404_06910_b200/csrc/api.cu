// Host-side pieces of the C ABI that launch nothing: error strings, layout checks,
// token position assignment, the device status read-back.
#include <cstring>

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
    return sp::fail(SP_ERR_CUDA, "unknown device status word %u", word);
}

}  // extern "C"
