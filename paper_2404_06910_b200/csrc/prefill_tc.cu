// Placeholder until the tensor-core kernel lands: bf16 / head_dim 128 runs the SIMT kernel.
#include "common.cuh"

namespace sp {
int launch_prefill_simt(const void *q, const void *k, const void *v, const sp_layout *lay, int n_heads,
                        int n_kv_heads, int head_dim, float scale, int rows, void *out, float *lse,
                        int dtype, cudaStream_t st);

size_t prefill_tc_workspace_bytes(int, int, int, int, int) { return 256; }

int launch_prefill_tc(const void *q, const void *k, const void *v, const sp_layout *lay, int n_heads,
                      int n_kv_heads, float scale, int rows, void *out, float *lse, void *ws,
                      size_t, cudaStream_t st)
{
    SP_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    return launch_prefill_simt(q, k, v, lay, n_heads, n_kv_heads, 128, scale, rows, out, lse, SP_BF16, st);
}
}  // namespace sp
