// sp_prune_topk: greedy top-k over each prompt's path scores and the softmax posterior
// at the kept paths (Section 3.2.3; Appendix B.1).
//
// Latency-sized: one warp per prompt.  Scores map to order-preserving 64-bit keys
// (score rank in the high word, reversed path index in the low word), so "largest key"
// gives descending score with ties to the lower index and NaN last; k rounds of a warp
// arg-max, each restricted to keys below the previous winner, select the k paths without
// any scratch memory or marking.
#include "common.cuh"

namespace sp {

// Monotone map float -> uint32: larger float => larger code; -0 == +0; NaN => 0.
__device__ __forceinline__ uint32_t order_code(float x)
{
    if (x != x) return 0u;
    if (x == 0.f) x = 0.f;                       // fold -0 onto +0
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w > v ? w : v;
    }
    return v;
}

__global__ void __launch_bounds__(128)
prune_topk_kernel(const float *__restrict__ scores, const int32_t *__restrict__ ppo, int n_prompts,
                  int k, int32_t *__restrict__ kept_idx, float *__restrict__ kept_post)
{
    const int b = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (b >= n_prompts) return;
    const int lane = threadIdx.x & 31;
    const int lo = ppo[b];
    const int n = max(ppo[b + 1] - lo, 0);

    float mx = -INFINITY, den = 0.f;
    if (kept_post) {                             // softmax statistics, NaN counted as -inf
        for (int i = lane; i < n; i += 32) {
            const float s = scores[lo + i];
            if (s == s) mx = fmaxf(mx, s);
        }
        mx = warp_max(mx);
        for (int i = lane; i < n; i += 32) {
            const float s = scores[lo + i];
            if (s == s && mx > -INFINITY) den += expf(s - mx);
        }
        den = warp_sum(den);
    }

    unsigned long long prev = ~0ull;             // every real key is below this
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;          // no real key is 0 (low word >= 1 below)
        if (j < n) {
            for (int i = lane; i < n; i += 32) {
                const unsigned long long key =
                    ((unsigned long long)order_code(scores[lo + i]) << 32) | (uint32_t)(0x7fffffff - i);
                if (key < prev && key > best) best = key;
            }
            best = warp_max_u64(best);
            prev = best;
        }
        if (lane == 0) {
            if (j < n) {
                const int i = 0x7fffffff - (int)(uint32_t)(best & 0xffffffffu);
                kept_idx[(int64_t)b * k + j] = lo + i;
                if (kept_post) {
                    const float s = scores[lo + i];
                    kept_post[(int64_t)b * k + j] = (s == s && den > 0.f) ? expf(s - mx) / den : 0.f;
                }
            } else {
                kept_idx[(int64_t)b * k + j] = -1;
                if (kept_post) kept_post[(int64_t)b * k + j] = 0.f;
            }
        }
    }
}

}  // namespace sp

extern "C" int sp_prune_topk(const float *scores, const int32_t *prompt_path_off, int n_prompts,
                             int k, int32_t *kept_idx, float *kept_post, void *stream)
{
    using namespace sp;
    SP_REQUIRE(k >= 1, SP_ERR_INVALID_ARG, "sp_prune_topk: k must be >= 1 (got %d)", k);
    SP_REQUIRE(n_prompts >= 0, SP_ERR_INVALID_ARG, "sp_prune_topk: n_prompts < 0");
    if (n_prompts == 0) return SP_OK;
    SP_REQUIRE(scores && prompt_path_off && kept_idx, SP_ERR_INVALID_ARG, "sp_prune_topk: NULL pointer");
    prune_topk_kernel<<<(n_prompts + 3) / 4, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        scores, prompt_path_off, n_prompts, k, kept_idx, kept_post);
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}
