// sp_rope_apply: rotary position encoding at real-valued positions (Section 3.2.2,
// footnote on RoPE: the sinusoid's argument is evaluated at the interpolated position).
//
// HBM-bound: one read and one write of x.  The rot_dim/2 angles of a token are the same
// for all of its heads, so each (token, pair) angle is evaluated once, in fp64, by one
// thread and shared through shared memory; the data pass is 16-byte vector loads/stores.
#include "common.cuh"

namespace sp {

struct RopeFreq {
    double inv_freq[128];   // base^(-2m/rot_dim), m < rot_dim/2 <= 128, computed on the host
};

constexpr int kRopeThreads = 256;
constexpr int kRopeTokens = 4;   // tokens per block iteration

template <typename T> struct Pack;
template <> struct Pack<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16 *p, float (&f)[8]) { Vec<__nv_bfloat16>::load(p, f); }
    __device__ static void store(__nv_bfloat16 *p, const float (&f)[8]) {
        uint4 w;
        w.x = pack_bf16x2(f[0], f[1]); w.y = pack_bf16x2(f[2], f[3]);
        w.z = pack_bf16x2(f[4], f[5]); w.w = pack_bf16x2(f[6], f[7]);
        *reinterpret_cast<uint4 *>(p) = w;
    }
};
template <> struct Pack<float> {
    static constexpr int N = 4;
    __device__ static void load(const float *p, float (&f)[4]) { Vec<float>::load(p, f); }
    __device__ static void store(float *p, const float (&f)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
    }
};

// Rotates nt tokens (starting at t0) of one tensor with the (cos, sin) table of the group.
// VEC: 16-byte accesses (requires alignment and divisibility, checked by the host).
template <typename T, bool VEC>
__device__ __forceinline__ void rotate_tokens(T *__restrict__ x, const float2 (*cs)[128], int64_t t0, int nt,
                                              int64_t ld_token, int n_heads, int head_dim, int rot_dim, int pairing)
{
    const int half = rot_dim >> 1;
    if (VEC) {
        constexpr int N = Pack<T>::N;
        if (pairing == SP_ROPE_HALF_SPLIT) {
            const int vec_per_head = half / N;
            const int items = nt * n_heads * vec_per_head;
            for (int i = threadIdx.x; i < items; i += kRopeThreads) {
                const int t = i / (n_heads * vec_per_head);
                const int r = i - t * (n_heads * vec_per_head);
                const int h = r / vec_per_head, m0 = (r - h * vec_per_head) * N;
                T *pa = x + (t0 + t) * ld_token + (int64_t)h * head_dim + m0;
                T *pb = pa + half;
                float a[N], b[N];
                Pack<T>::load(pa, a);
                Pack<T>::load(pb, b);
#pragma unroll
                for (int j = 0; j < N; ++j) {
                    const float2 w = cs[t][m0 + j];
                    rope_rotate(a[j], b[j], w.x, w.y, a[j], b[j]);
                }
                Pack<T>::store(pa, a);
                Pack<T>::store(pb, b);
            }
        } else {
            const int vec_per_head = rot_dim / N;
            const int items = nt * n_heads * vec_per_head;
            for (int i = threadIdx.x; i < items; i += kRopeThreads) {
                const int t = i / (n_heads * vec_per_head);
                const int r = i - t * (n_heads * vec_per_head);
                const int h = r / vec_per_head, e0 = (r - h * vec_per_head) * N;
                T *p = x + (t0 + t) * ld_token + (int64_t)h * head_dim + e0;
                float f[N];
                Pack<T>::load(p, f);
#pragma unroll
                for (int j = 0; j < N; j += 2) {
                    const float2 w = cs[t][(e0 + j) >> 1];
                    rope_rotate(f[j], f[j + 1], w.x, w.y, f[j], f[j + 1]);
                }
                Pack<T>::store(p, f);
            }
        }
    } else {
        const int items = nt * n_heads * half;
        for (int i = threadIdx.x; i < items; i += kRopeThreads) {
            const int t = i / (n_heads * half);
            const int r = i - t * (n_heads * half);
            const int h = r / half, m = r - h * half;
            T *base = x + (t0 + t) * ld_token + (int64_t)h * head_dim;
            T *pa = base + (pairing == SP_ROPE_HALF_SPLIT ? m : 2 * m);
            T *pb = base + (pairing == SP_ROPE_HALF_SPLIT ? m + half : 2 * m + 1);
            const float a = to_float(*pa), b = to_float(*pb);
            const float2 w = cs[t][m];
            float na, nb;
            rope_rotate(a, b, w.x, w.y, na, nb);
            store_val(pa, na);
            store_val(pb, nb);
        }
    }
}

// One launch may rotate two tensors that share their positions (a step's Q and K): x1 == NULL
// rotates x alone.  VEC / VEC1: whether the 16-byte path applies to x / x1.
template <typename T, bool VEC, bool VEC1>
__global__ void __launch_bounds__(kRopeThreads, 8)   // 32 registers: full occupancy for the streaming pass
rope_kernel(T *__restrict__ x, T *__restrict__ x1, const float *__restrict__ pos, int64_t n_tokens, int64_t ld_token,
            int64_t ld_token1, int n_heads, int n_heads1, int head_dim, int rot_dim, int pairing,
            const __grid_constant__ RopeFreq fr)
{
    __shared__ float2 cs[kRopeTokens][128];   // (cos, sin) per (token, pair)
    const int half = rot_dim >> 1;
    const int64_t n_groups = (n_tokens + kRopeTokens - 1) / kRopeTokens;

    for (int64_t g = blockIdx.x; g < n_groups; g += gridDim.x) {
        const int64_t t0 = g * kRopeTokens;
        const int nt = (int)min((int64_t)kRopeTokens, n_tokens - t0);
        __syncthreads();
        for (int i = threadIdx.x; i < nt * half; i += kRopeThreads) {
            const int t = i / half, m = i - t * half;
            double s, c;
            sincos((double)pos[t0 + t] * fr.inv_freq[m], &s, &c);
            cs[t][m] = make_float2((float)c, (float)s);
        }
        __syncthreads();
        rotate_tokens<T, VEC>(x, cs, t0, nt, ld_token, n_heads, head_dim, rot_dim, pairing);
        if (x1) rotate_tokens<T, VEC1>(x1, cs, t0, nt, ld_token1, n_heads1, head_dim, rot_dim, pairing);
    }
}

template <typename T>
static bool rope_vec_ok(const void *x, int64_t ld_token, int head_dim, int rot_dim, int pairing)
{
    constexpr int N = Pack<T>::N;
    const int half = rot_dim / 2;
    return aligned16(x) && (ld_token % N == 0) && (head_dim % N == 0) &&
           (pairing == SP_ROPE_HALF_SPLIT ? (half % N == 0) : (rot_dim % N == 0));
}

template <typename T>
static int launch_rope(void *x, void *x1, const float *pos, int64_t n_tokens, int64_t ld_token, int64_t ld_token1,
                       int n_heads, int n_heads1, int head_dim, int rot_dim, int pairing, const RopeFreq &fr,
                       cudaStream_t st)
{
    const bool v0 = rope_vec_ok<T>(x, ld_token, head_dim, rot_dim, pairing);
    const bool v1 = x1 == nullptr || rope_vec_ok<T>(x1, ld_token1, head_dim, rot_dim, pairing);
    const int64_t n_groups = (n_tokens + kRopeTokens - 1) / kRopeTokens;
    const int grid = (int)std::min<int64_t>(n_groups, (int64_t)num_sms() * 16);
    auto go = [&](auto kern) {
        kern<<<grid, kRopeThreads, 0, st>>>((T *)x, (T *)x1, pos, n_tokens, ld_token, ld_token1, n_heads, n_heads1,
                                            head_dim, rot_dim, pairing, fr);
    };
    if (v0 && v1) go(rope_kernel<T, true, true>);
    else if (v0) go(rope_kernel<T, true, false>);
    else if (v1) go(rope_kernel<T, false, true>);
    else go(rope_kernel<T, false, false>);
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

static int rope_entry(const char *name, void *x, int64_t ld_token, int n_heads, void *x1, int64_t ld_token1, int n_heads1,
                      const float *pos, int64_t n_tokens, int head_dim, int rot_dim, double base, int pairing,
                      int dtype, void *stream)
{
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "%s: unknown dtype %d", name, dtype);
    SP_REQUIRE(n_tokens >= 0, SP_ERR_INVALID_ARG, "%s: n_tokens < 0", name);
    SP_REQUIRE(n_heads > 0 && head_dim > 0 && head_dim <= 256 && (x1 == nullptr || n_heads1 > 0), SP_ERR_INVALID_ARG,
               "%s: n_heads %d / %d / head_dim %d out of range", name, n_heads, n_heads1, head_dim);
    SP_REQUIRE(rot_dim >= 2 && rot_dim <= head_dim && (rot_dim & 1) == 0, SP_ERR_INVALID_ARG,
               "%s: rot_dim %d must be even and in [2, head_dim]", name, rot_dim);
    SP_REQUIRE(pairing == SP_ROPE_HALF_SPLIT || pairing == SP_ROPE_INTERLEAVED, SP_ERR_INVALID_ARG,
               "%s: unknown pairing %d", name, pairing);
    SP_REQUIRE(ld_token >= (int64_t)n_heads * head_dim && (x1 == nullptr || ld_token1 >= (int64_t)n_heads1 * head_dim),
               SP_ERR_INVALID_ARG, "%s: ld_token < n_heads*head_dim", name);
    SP_REQUIRE(base > 0.0, SP_ERR_INVALID_ARG, "%s: base must be positive", name);
    if (n_tokens == 0) return SP_OK;
    SP_REQUIRE(x != nullptr && pos != nullptr, SP_ERR_INVALID_ARG, "%s: NULL pointer", name);
    SP_REQUIRE((reinterpret_cast<uintptr_t>(x) % elt_bytes(dtype)) == 0 &&
                   (reinterpret_cast<uintptr_t>(x1) % elt_bytes(dtype)) == 0,
               SP_ERR_INVALID_ARG, "%s: x is not aligned to its element size", name);

    RopeFreq fr;
    for (int m = 0; m < rot_dim / 2; ++m) fr.inv_freq[m] = std::pow(base, -2.0 * m / rot_dim);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return dtype == SP_F32
               ? launch_rope<float>(x, x1, pos, n_tokens, ld_token, ld_token1, n_heads, n_heads1, head_dim, rot_dim, pairing, fr, st)
               : launch_rope<__nv_bfloat16>(x, x1, pos, n_tokens, ld_token, ld_token1, n_heads, n_heads1, head_dim, rot_dim, pairing, fr, st);
}

// The (cos, sin) of every (token, pair) as a table in device memory, for kernels that rotate tiles on the fly:
// the same fp64 evaluation as above, so a tile rotated from the table equals one rotated by rope_kernel.
__global__ void __launch_bounds__(256) rope_table_kernel(const float *__restrict__ pos, int64_t n_tokens, int half,
                                                          float2 *__restrict__ out, const __grid_constant__ RopeFreq fr)
{
    const int64_t n = n_tokens * half;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i / half;
        const int m = (int)(i - t * half);
        double s, c;
        sincos((double)pos[t] * fr.inv_freq[m], &s, &c);
        out[i] = make_float2((float)c, (float)s);
    }
}

int launch_rope_table(const float *pos, int64_t n_tokens, int rot_dim, double base, float2 *out, cudaStream_t st)
{
    if (n_tokens <= 0) return SP_OK;
    RopeFreq fr;
    for (int m = 0; m < rot_dim / 2; ++m) fr.inv_freq[m] = std::pow(base, -2.0 * m / rot_dim);
    const int64_t n = n_tokens * (rot_dim / 2);
    const int grid = (int)std::min<int64_t>((n + 255) / 256, (int64_t)num_sms() * 16);
    rope_table_kernel<<<grid, 256, 0, st>>>(pos, n_tokens, rot_dim / 2, out, fr);
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

}  // namespace sp

extern "C" int sp_rope_apply(void *x, const float *pos, int64_t n_tokens, int64_t ld_token,
                             int n_heads, int head_dim, int rot_dim, double base, int pairing,
                             int dtype, void *stream)
{
    return sp::rope_entry("sp_rope_apply", x, ld_token, n_heads, nullptr, 0, 0, pos, n_tokens, head_dim, rot_dim, base,
                          pairing, dtype, stream);
}

extern "C" int sp_rope_apply_pair(void *xq, int64_t ld_q, int n_heads_q, void *xk, int64_t ld_k, int n_heads_k,
                                  const float *pos, int64_t n_tokens, int head_dim, int rot_dim, double base,
                                  int pairing, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(n_tokens == 0 || xk != nullptr, SP_ERR_INVALID_ARG, "sp_rope_apply_pair: NULL pointer");
    return rope_entry("sp_rope_apply_pair", xq, ld_q, n_heads_q, xk, ld_k, n_heads_k, pos, n_tokens, head_dim, rot_dim,
                      base, pairing, dtype, stream);
}
