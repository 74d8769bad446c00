// Fork-join prefill attention, fp32 SIMT variant (Section 3.2: a row attends to its
// prompt's preamble and, causally, to its own path).
//
// Used where the tensor-core kernel does not apply: fp32 storage (tight tolerance rules
// out reduced-precision products) and head_dim 64.  One warp owns one (row, head): the
// head dimension is spread over the lanes, scores are warp-reduced, softmax is online
// with exact exp2f.  Masked keys are never visited: the loop runs over the row's key
// ranges only.
#include "common.cuh"

namespace sp {

constexpr int kSimtWarps = 8;
constexpr float kLog2eP = 1.4426950408889634f;
constexpr float kLn2P = 0.6931471805599453f;

struct PrefillSimtArgs {
    const void *q, *k, *v;
    void *out;
    float *lse;
    const int32_t *ppo, *pre_start, *pre_len, *path_start, *doc_len, *qry_len;
    int n_prompts, n_paths, n_heads, n_kv_heads, rows_mode;
    int64_t total_tokens;
    float scale_log2e;
    const float *pos, *slopes;   // ALiBi: token positions [T] and head slopes [H]; NULL = no bias
};

template <typename T, int EPL> struct LaneVec;     // EPL contiguous elements of one lane
template <> struct LaneVec<float, 2> {
    __device__ static void load(const float *p, float (&f)[2]) { const float2 w = *reinterpret_cast<const float2 *>(p); f[0] = w.x; f[1] = w.y; }
    __device__ static void store(float *p, const float (&f)[2]) { *reinterpret_cast<float2 *>(p) = make_float2(f[0], f[1]); }
};
template <> struct LaneVec<float, 4> {
    __device__ static void load(const float *p, float (&f)[4]) { const float4 w = *reinterpret_cast<const float4 *>(p); f[0] = w.x; f[1] = w.y; f[2] = w.z; f[3] = w.w; }
    __device__ static void store(float *p, const float (&f)[4]) { *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]); }
};
template <> struct LaneVec<__nv_bfloat16, 2> {
    __device__ static void load(const __nv_bfloat16 *p, float (&f)[2]) { const uint32_t w = *reinterpret_cast<const uint32_t *>(p); f[0] = bf16_lo(w); f[1] = bf16_hi(w); }
    __device__ static void store(__nv_bfloat16 *p, const float (&f)[2]) { *reinterpret_cast<uint32_t *>(p) = pack_bf16x2(f[0], f[1]); }
};
template <> struct LaneVec<__nv_bfloat16, 4> {
    __device__ static void load(const __nv_bfloat16 *p, float (&f)[4]) { const uint2 w = *reinterpret_cast<const uint2 *>(p); f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y); }
    __device__ static void store(__nv_bfloat16 *p, const float (&f)[4]) { *reinterpret_cast<uint2 *>(p) = make_uint2(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3])); }
};

// grid: x = sequence (prompt preambles first, then paths), y = head.
template <typename T, int D>
__global__ void __launch_bounds__(kSimtWarps * 32)
prefill_simt_kernel(const __grid_constant__ PrefillSimtArgs a)
{
    constexpr int EPL = D / 32;
    const int seq = blockIdx.x, h = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hk = h / (a.n_heads / a.n_kv_heads);

    // key ranges of this sequence: [pre_lo, pre_lo+pre_n) fully visible, own rows causal
    int pre_lo, pre_n, own_lo, own_n, first_row;
    if (seq < a.n_prompts) {
        if (a.rows_mode == SP_ROWS_QUERY_ONLY) return;
        pre_lo = 0; pre_n = 0;
        own_lo = a.pre_start[seq]; own_n = a.pre_len[seq]; first_row = 0;
    } else {
        const int i = seq - a.n_prompts;
        int lo = 0, hi = a.n_prompts - 1;           // prompt owning path i
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (a.ppo[mid] <= i) lo = mid; else hi = mid - 1;
        }
        pre_lo = a.pre_start[lo]; pre_n = a.pre_len[lo];
        own_lo = a.path_start[i]; own_n = a.doc_len[i] + a.qry_len[i];
        first_row = a.rows_mode == SP_ROWS_QUERY_ONLY ? a.doc_len[i] : 0;
    }

    const T *Q = static_cast<const T *>(a.q);
    const T *K = static_cast<const T *>(a.k) + (int64_t)hk * D + lane * EPL;
    const T *V = static_cast<const T *>(a.v) + (int64_t)hk * D + lane * EPL;
    const int64_t kv_stride = (int64_t)a.n_kv_heads * D;

    for (int j = first_row + warp; j < own_n; j += kSimtWarps) {
        const int64_t r = own_lo + j;
        float qf[EPL], acc[EPL];
        LaneVec<T, EPL>::load(Q + (r * a.n_heads + h) * D + lane * EPL, qf);
#pragma unroll
        for (int e = 0; e < EPL; ++e) { qf[e] *= a.scale_log2e; acc[e] = 0.f; }
        float m = -INFINITY, l = 0.f;
        const float pq = a.pos ? a.pos[r] : 0.f;
        const float slope_l2 = a.pos ? a.slopes[h] * kLog2eP : 0.f;

        const int n_keys = pre_n + j + 1;
        for (int c = 0; c < n_keys; ++c) {
            const int64_t kr = c < pre_n ? (int64_t)pre_lo + c : (int64_t)own_lo + (c - pre_n);
            float kf[EPL], vf[EPL];
            LaneVec<T, EPL>::load(K + kr * kv_stride, kf);
            LaneVec<T, EPL>::load(V + kr * kv_stride, vf);
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) s = fmaf(qf[e], kf[e], s);
            s = warp_sum(s);
            if (a.pos) s -= slope_l2 * fabsf(pq - a.pos[kr]);     // ALiBi: linear distance penalty
            if (s > m) {
                const float rs = exp2f(m - s);
                l *= rs;
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[e] *= rs;
                m = s;
            }
            const float p = exp2f(s - m);
            l += p;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
        }
        const float inv = 1.f / l;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= inv;
        LaneVec<T, EPL>::store(static_cast<T *>(a.out) + (r * a.n_heads + h) * D + lane * EPL, acc);
        if (a.lse && lane == 0) a.lse[(int64_t)h * a.total_tokens + r] = (m + log2f(l)) * kLn2P;
    }
}

int launch_prefill_simt(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                        const float *slopes, int n_heads, int n_kv_heads, int head_dim, float scale, int rows,
                        void *out, float *lse, int dtype, cudaStream_t st)
{
    PrefillSimtArgs a;
    a.q = q; a.k = k; a.v = v; a.out = out; a.lse = lse;
    a.ppo = lay->prompt_path_off; a.pre_start = lay->pre_start; a.pre_len = lay->pre_len;
    a.path_start = lay->path_start; a.doc_len = lay->doc_len; a.qry_len = lay->qry_len;
    a.n_prompts = lay->n_prompts; a.n_paths = lay->n_paths; a.n_heads = n_heads; a.n_kv_heads = n_kv_heads;
    a.rows_mode = rows; a.total_tokens = lay->total_tokens; a.scale_log2e = scale * kLog2eP;
    a.pos = pos; a.slopes = slopes;
    const dim3 grid(lay->n_prompts + lay->n_paths, n_heads);
    const int threads = kSimtWarps * 32;
    if (dtype == SP_F32) {
        if (head_dim == 64) prefill_simt_kernel<float, 64><<<grid, threads, 0, st>>>(a);
        else                prefill_simt_kernel<float, 128><<<grid, threads, 0, st>>>(a);
    } else {
        if (head_dim == 64) prefill_simt_kernel<__nv_bfloat16, 64><<<grid, threads, 0, st>>>(a);
        else                prefill_simt_kernel<__nv_bfloat16, 128><<<grid, threads, 0, st>>>(a);
    }
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

}  // namespace sp
