// sp_path_scores: Bayesian path saliency (Section 3.2.3; Appendix B.1, Eq. 2).
//
// The logits tensor [paths * query length, vocab] is the largest object of the online
// phase and each element is needed exactly once, so the kernel is one streaming HBM
// pass: a block per scored row, 16-byte cache-streaming loads, a per-thread online
// (max, sum of exponentials) pair merged by warp shuffles, one log per row.  Rows whose
// target is -1 are not read at all.  A second tiny kernel adds each path's rows in a
// fixed order (no float atomics), so scores are reproducible bit for bit.
#include "common.cuh"

namespace sp {

constexpr int kScoreThreads = 256;
constexpr int kScoreUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Merges (m2, s2) into (m, s): s counts exponentials relative to the running maximum m.
__device__ __forceinline__ void merge_ms(float &m, float &s, float m2, float s2)
{
    const float mn = fmaxf(m, m2);
    const float a = (m == mn) ? 1.f : fast_exp2((m - mn) * kLog2e);     // also covers m == -inf
    const float b = (m2 == mn) ? 1.f : fast_exp2((m2 - mn) * kLog2e);
    s = s * a + s2 * b;
    m = mn;
}

template <typename T> __device__ __forceinline__ void load_stream(const T *p, float (&f)[Vec<T>::N]);
template <> __device__ __forceinline__ void load_stream<__nv_bfloat16>(const __nv_bfloat16 *p, float (&f)[8])
{
    const uint4 w = __ldcs(reinterpret_cast<const uint4 *>(p));
    f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
    f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
}
template <> __device__ __forceinline__ void load_stream<float>(const float *p, float (&f)[4])
{
    const float4 w = __ldcs(reinterpret_cast<const float4 *>(p));
    f[0] = w.x; f[1] = w.y; f[2] = w.z; f[3] = w.w;
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(kScoreThreads)
row_logp_kernel(const T *__restrict__ logits, int64_t ld, const int32_t *__restrict__ targets,
                int vocab, float *__restrict__ row_logp)
{
    const int64_t t = blockIdx.x;
    const int32_t y = targets[t];
    if (y < 0 || y >= vocab) {           // no target: contributes nothing, row is not read
        if (threadIdx.x == 0) row_logp[t] = 0.f;
        return;
    }
    const T *row = logits + t * ld;
    float m = -INFINITY, s = 0.f;

    constexpr int N = Vec<T>::N;
    int done = 0;
    if (VEC) {
        const int nvec = vocab / N;
        for (int i0 = threadIdx.x; i0 < nvec; i0 += kScoreThreads * kScoreUnroll) {
            float f[kScoreUnroll][N];
#pragma unroll
            for (int u = 0; u < kScoreUnroll; ++u) {
                const int i = i0 + u * kScoreThreads;
                if (i < nvec) {
                    load_stream<T>(row + (int64_t)i * N, f[u]);
                } else {
#pragma unroll
                    for (int j = 0; j < N; ++j) f[u][j] = -INFINITY;
                }
            }
            float cm = f[0][0];
#pragma unroll
            for (int u = 0; u < kScoreUnroll; ++u)
#pragma unroll
                for (int j = 0; j < N; ++j) cm = fmaxf(cm, f[u][j]);
            if (cm > m) {                 // rescale the running sum to the new maximum
                s *= fast_exp2((m - cm) * kLog2e);
                m = cm;
            }
            const float mb = m * kLog2e;
            float acc = 0.f;
#pragma unroll
            for (int u = 0; u < kScoreUnroll; ++u)
#pragma unroll
                for (int j = 0; j < N; ++j) acc += fast_exp2(fmaf(f[u][j], kLog2e, -mb));
            s += acc;
        }
        done = nvec * N;
    }
    for (int c = done + threadIdx.x; c < vocab; c += kScoreThreads) {   // tail / unaligned rows
        const float xv = to_float(row[c]);
        if (xv > m) { s *= fast_exp2((m - xv) * kLog2e); m = xv; }
        s += fast_exp2((xv - m) * kLog2e);
    }

#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
        merge_ms(m, s, m2, s2);
    }
    __shared__ float sm[kScoreThreads / 32], ss[kScoreThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { sm[warp] = m; ss[warp] = s; }
    __syncthreads();
    if (threadIdx.x == 0) {
        m = sm[0]; s = ss[0];
        for (int w = 1; w < kScoreThreads / 32; ++w) merge_ms(m, s, sm[w], ss[w]);
        row_logp[t] = to_float(row[y]) - (m + logf(s));
    }
}

// scores[i] = weight[i] * sum_t row_logp[t] + prior[i]; one warp per path, fixed order.
__global__ void __launch_bounds__(256)
path_sum_kernel(const float *__restrict__ row_logp, const int32_t *__restrict__ row_off, int n_paths,
                const float *__restrict__ prior, const float *__restrict__ weight,
                float *__restrict__ scores)
{
    const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (i >= n_paths) return;
    const int lane = threadIdx.x & 31;
    double acc = 0.0;
    for (int t = row_off[i] + lane; t < row_off[i + 1]; t += 32) acc += (double)row_logp[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
        const double w = weight ? (double)weight[i] : 1.0;
        const double pr = prior ? (double)prior[i] : 0.0;
        scores[i] = (float)(w * acc + pr);
    }
}

}  // namespace sp

extern "C" size_t sp_path_scores_workspace_bytes(int64_t n_rows)
{
    return sp::round_up(256 + (size_t)(n_rows > 0 ? n_rows : 0) * sizeof(float), 256);
}

extern "C" int sp_path_scores(const void *logits, int64_t ld_logits, const int32_t *targets,
                              const int32_t *row_off, int64_t n_rows, int n_paths, int vocab,
                              const float *prior, const float *weight, float *scores,
                              float *row_logp, void *ws, size_t ws_bytes, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "sp_path_scores: unknown dtype %d", dtype);
    SP_REQUIRE(n_rows >= 0 && n_rows < (int64_t)INT32_MAX && n_paths >= 0, SP_ERR_INVALID_ARG,
               "sp_path_scores: n_rows %lld / n_paths %d out of range", (long long)n_rows, n_paths);
    SP_REQUIRE(vocab > 0 && ld_logits >= vocab, SP_ERR_INVALID_ARG,
               "sp_path_scores: vocab %d must be positive and <= ld_logits %lld", vocab, (long long)ld_logits);
    if (n_paths == 0) return SP_OK;
    SP_REQUIRE(row_off && scores, SP_ERR_INVALID_ARG, "sp_path_scores: row_off / scores is NULL");
    SP_REQUIRE(n_rows == 0 || (logits && targets), SP_ERR_INVALID_ARG, "sp_path_scores: logits / targets is NULL");
    SP_REQUIRE((reinterpret_cast<uintptr_t>(logits) % elt_bytes(dtype)) == 0, SP_ERR_INVALID_ARG,
               "sp_path_scores: logits not aligned to the element size");
    float *rows_out = row_logp;
    if (!rows_out) {
        SP_REQUIRE(ws && aligned256(ws) && ws_bytes >= sp_path_scores_workspace_bytes(n_rows), SP_ERR_WORKSPACE,
                   "sp_path_scores: workspace of %zu bytes (256-byte aligned) required when row_logp is NULL",
                   sp_path_scores_workspace_bytes(n_rows));
        rows_out = reinterpret_cast<float *>(static_cast<char *>(ws) + 256);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_rows > 0) {
        const bool vec = aligned16(logits) && ((ld_logits * elt_bytes(dtype)) % 16 == 0);
        const unsigned grid = (unsigned)n_rows;
        if (dtype == SP_BF16) {
            auto *p = static_cast<const __nv_bfloat16 *>(logits);
            if (vec) row_logp_kernel<__nv_bfloat16, true><<<grid, kScoreThreads, 0, st>>>(p, ld_logits, targets, vocab, rows_out);
            else     row_logp_kernel<__nv_bfloat16, false><<<grid, kScoreThreads, 0, st>>>(p, ld_logits, targets, vocab, rows_out);
        } else {
            auto *p = static_cast<const float *>(logits);
            if (vec) row_logp_kernel<float, true><<<grid, kScoreThreads, 0, st>>>(p, ld_logits, targets, vocab, rows_out);
            else     row_logp_kernel<float, false><<<grid, kScoreThreads, 0, st>>>(p, ld_logits, targets, vocab, rows_out);
        }
        SP_CUDA(cudaGetLastError());
    }
    path_sum_kernel<<<(n_paths + 7) / 8, 256, 0, st>>>(rows_out, row_off, n_paths, prior, weight, scores);
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}
