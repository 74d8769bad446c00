// sp_superpose_prefill entry point: argument checks and kernel selection.
#include <algorithm>

#include "common.cuh"

namespace sp {
int launch_prefill_simt(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                        const float *slopes, int n_heads, int n_kv_heads, int head_dim, float scale, int rows,
                        void *out, float *lse, int dtype, cudaStream_t st);
size_t prefill_tc_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len, int n_heads);
int launch_prefill_tc(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                      const float *slopes, int n_heads, int n_kv_heads, float scale, int rows, void *out,
                      float *lse, void *ws, size_t ws_bytes, cudaStream_t st);
size_t prefill_tc_rope_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len, int64_t total_tokens);
int launch_prefill_tc_rope(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos, double base,
                           int pairing, int n_heads, int n_kv_heads, float scale, void *out, float *lse, void *ws,
                           cudaStream_t st);
size_t prefill_qonly_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len);
int launch_prefill_qonly(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                         const float *slopes, int n_heads, int n_kv_heads, float scale, void *out, float *lse,
                         void *ws, cudaStream_t st);
}  // namespace sp

extern "C" size_t sp_prefill_workspace_bytes(int n_prompts, int n_paths, int max_pre_len,
                                             int max_path_len, int n_heads, int head_dim, int dtype)
{
    if (dtype == SP_BF16 && head_dim == 128)      // enough for either rows mode
        return std::max(sp::prefill_tc_workspace_bytes(n_prompts, n_paths, max_pre_len, max_path_len, n_heads),
                        sp::prefill_qonly_workspace_bytes(n_prompts, n_paths, max_pre_len, max_path_len));
    return 256;
}

namespace sp {
static int prefill_entry(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                         const float *slopes, int n_heads, int n_kv_heads, int head_dim, float scale, int rows,
                         void *out, float *lse, void *ws, size_t ws_bytes, int dtype, void *stream)
{
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "sp_superpose_prefill: unknown dtype %d", dtype);
    if (int rc = check_layout(lay)) return rc;
    SP_REQUIRE(head_dim == 64 || head_dim == 128, SP_ERR_UNSUPPORTED,
               "sp_superpose_prefill: head_dim %d (64 or 128 supported)", head_dim);
    SP_REQUIRE(n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0 && n_heads <= 65535, SP_ERR_INVALID_ARG,
               "sp_superpose_prefill: n_heads %d must be a positive multiple of n_kv_heads %d", n_heads, n_kv_heads);
    SP_REQUIRE(rows == SP_ROWS_ALL || rows == SP_ROWS_QUERY_ONLY, SP_ERR_INVALID_ARG,
               "sp_superpose_prefill: unknown rows mode %d", rows);
    SP_REQUIRE(scale == scale && scale > 0.f, SP_ERR_INVALID_ARG, "sp_superpose_prefill: scale must be positive");
    if (lay->total_tokens == 0 || lay->n_prompts == 0) return SP_OK;
    SP_REQUIRE(q && k && v && out, SP_ERR_INVALID_ARG, "sp_superpose_prefill: NULL tensor");
    SP_REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(out), SP_ERR_INVALID_ARG,
               "sp_superpose_prefill: tensors must be 16-byte aligned");
    const size_t need = sp_prefill_workspace_bytes(lay->n_prompts, lay->n_paths, lay->max_pre_len,
                                                   lay->max_path_len, n_heads, head_dim, dtype);
    SP_REQUIRE(ws && aligned256(ws) && ws_bytes >= need, SP_ERR_WORKSPACE,
               "sp_superpose_prefill: workspace of %zu bytes (256-byte aligned) required", need);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == SP_BF16 && head_dim == 128 && rows == SP_ROWS_QUERY_ONLY)
        return launch_prefill_qonly(q, k, v, lay, pos, slopes, n_heads, n_kv_heads, scale, out, lse, ws, st);
    if (dtype == SP_BF16 && head_dim == 128)
        return launch_prefill_tc(q, k, v, lay, pos, slopes, n_heads, n_kv_heads, scale, rows, out, lse, ws, ws_bytes, st);
    SP_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    return launch_prefill_simt(q, k, v, lay, pos, slopes, n_heads, n_kv_heads, head_dim, scale, rows, out, lse, dtype, st);
}
}  // namespace sp

extern "C" int sp_superpose_prefill(const void *q, const void *k, const void *v, const sp_layout *lay,
                                    int n_heads, int n_kv_heads, int head_dim, float scale, int rows,
                                    void *out, float *lse, void *ws, size_t ws_bytes, int dtype,
                                    void *stream)
{
    return sp::prefill_entry(q, k, v, lay, nullptr, nullptr, n_heads, n_kv_heads, head_dim, scale, rows, out, lse,
                             ws, ws_bytes, dtype, stream);
}

extern "C" int sp_superpose_prefill_alibi(const void *q, const void *k, const void *v, const sp_layout *lay,
                                          const float *pos, const float *slopes, int n_heads, int n_kv_heads,
                                          int head_dim, float scale, int rows, void *out, float *lse, void *ws,
                                          size_t ws_bytes, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(lay == nullptr || lay->total_tokens == 0 || (pos && slopes), SP_ERR_INVALID_ARG,
               "sp_superpose_prefill_alibi: pos and slopes are required");
    return prefill_entry(q, k, v, lay, pos, slopes, n_heads, n_kv_heads, head_dim, scale, rows, out, lse, ws,
                         ws_bytes, dtype, stream);
}

extern "C" size_t sp_prefill_rope_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len,
                                                  int64_t total_tokens, int n_heads, int head_dim, int dtype)
{
    (void)n_heads;
    if (dtype != SP_BF16 || head_dim != 128) return 256;
    return sp::prefill_tc_rope_workspace_bytes(n_prompts, n_paths, max_pre_len, max_path_len, total_tokens);
}

extern "C" int sp_superpose_prefill_rope(const void *q, const void *k, const void *v, const sp_layout *lay,
                                         const float *pos, double base, int pairing, int n_heads, int n_kv_heads,
                                         int head_dim, float scale, void *out, float *lse, void *ws, size_t ws_bytes,
                                         int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "sp_superpose_prefill_rope: unknown dtype %d", dtype);
    if (int rc = check_layout(lay)) return rc;
    SP_REQUIRE(n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0 && n_heads <= 65535, SP_ERR_INVALID_ARG,
               "sp_superpose_prefill_rope: n_heads %d must be a positive multiple of n_kv_heads %d", n_heads, n_kv_heads);
    SP_REQUIRE(pairing == SP_ROPE_HALF_SPLIT || pairing == SP_ROPE_INTERLEAVED, SP_ERR_INVALID_ARG,
               "sp_superpose_prefill_rope: unknown pairing %d", pairing);
    SP_REQUIRE(base > 0.0, SP_ERR_INVALID_ARG, "sp_superpose_prefill_rope: base must be positive");
    SP_REQUIRE(scale == scale && scale > 0.f, SP_ERR_INVALID_ARG, "sp_superpose_prefill_rope: scale must be positive");
    SP_REQUIRE(dtype == SP_BF16 && head_dim == 128, SP_ERR_UNSUPPORTED,
               "sp_superpose_prefill_rope: bf16 with head_dim 128 only (rotate with sp_rope_apply and call sp_superpose_prefill)");
    if (lay->total_tokens == 0 || lay->n_prompts == 0) return SP_OK;
    SP_REQUIRE(q && k && v && out && pos, SP_ERR_INVALID_ARG, "sp_superpose_prefill_rope: NULL pointer");
    SP_REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(out), SP_ERR_INVALID_ARG,
               "sp_superpose_prefill_rope: tensors must be 16-byte aligned");
    const size_t need = sp_prefill_rope_workspace_bytes(lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len,
                                                        lay->total_tokens, n_heads, head_dim, dtype);
    SP_REQUIRE(ws && aligned256(ws) && ws_bytes >= need, SP_ERR_WORKSPACE,
               "sp_superpose_prefill_rope: workspace of %zu bytes (256-byte aligned) required", need);
    return launch_prefill_tc_rope(q, k, v, lay, pos, base, pairing, n_heads, n_kv_heads, scale, out, lse, ws,
                                  static_cast<cudaStream_t>(stream));
}
