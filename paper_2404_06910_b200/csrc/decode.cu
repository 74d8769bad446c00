// sp_pruned_decode: one-token decode attention over the pruned cache (Section 3.2.3;
// Algorithm 3: preamble + kept (document + query) + task/response tokens).
//
// HBM-bound: every kept K and V row is read exactly once.  Pruning is an index list --
// the kernel walks [preamble | kept path ranges | tail] as one logical key sequence and
// never copies KV.  The sequence is split across blocks (split-KV) so that small batches
// still fill the machine; each block keeps an online softmax per key group, writes one
// partial (max, sum, unnormalised output), and the last block to finish a (prompt, head)
// merges the partials in split order, so results do not depend on scheduling.
#include "common.cuh"

namespace sp {

constexpr int kDecThreads = 128;
constexpr int kDecUnroll = 4;        // keys in flight per key group (kept small: occupancy hides latency better)
constexpr int kDecMaxSplits = 64;
constexpr float kLog2eD = 1.4426950408889634f;
constexpr float kLn2D = 0.6931471805599453f;

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct DecodeArgs {
    const void *q, *k_cache, *v_cache, *tail_k, *tail_v;
    const int32_t *ppo, *pre_start, *pre_len, *path_start, *doc_len, *qry_len;
    const int32_t *kept_idx, *tail_len;
    void *out;
    float *lse;
    float *partial;          // [B*H][n_splits][D+2]
    unsigned int *counters;  // [B*H], zero on entry
    int k, tail_cap, n_heads, n_kv_heads, n_splits;
    float scale_log2e;
    // ALiBi variant only: positions of the query token [B], of the cache rows [T] and of the
    // tail rows [B, tail_cap], and the per-head slopes [H]
    const float *q_pos, *cache_pos, *tail_pos, *slopes;
};

// Workspace layout: [0,256) status word | counters [B*H] u32 | partials.
static size_t decode_counter_bytes(int n_prompts, int n_heads)
{
    return round_up((size_t)n_prompts * n_heads * sizeof(unsigned int), 256);
}
static int decode_split_cap(int n_prompts, int n_heads)
{
    const int64_t bh = std::max<int64_t>(1, (int64_t)n_prompts * n_heads);
    const int64_t want = (8LL * kNumSMs) / bh;      // 8 blocks per SM: all blocks of a launch are resident at once
    return (int)std::min<int64_t>(kDecMaxSplits, std::max<int64_t>(1, want));
}

// 16 bytes of a key / value row, kept raw until the arithmetic needs them.
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 w;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "l"(p));
    return w;
}
template <typename T> struct Raw16;
template <> struct Raw16<__nv_bfloat16> {
    __device__ __forceinline__ static void unpack(const uint4 &w, float (&f)[8]) {
        f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
        f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
    }
};
template <> struct Raw16<float> {
    __device__ __forceinline__ static void unpack(const uint4 &w, float (&f)[4]) {
        f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y); f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
    }
};

// ALIBI: scores get -slope_h * |pos_q - pos_k| (Section 3.2.2: real-valued positions pose no
// problem for ALiBi); the plain instantiation carries none of that code.
template <typename T, int D, bool ALIBI>
__global__ void __launch_bounds__(kDecThreads, 8)
decode_kernel(const __grid_constant__ DecodeArgs a)
{
    constexpr int N = Vec<T>::N;            // elements per 16-byte load
    constexpr int LPK = D / N;              // lanes that share one key row
    constexpr int G = kDecThreads / LPK;    // key groups per block
    static_assert(LPK <= 32 && (32 % LPK) == 0, "a key row must fit in one warp");

    extern __shared__ __align__(16) unsigned char smem_raw[];
    // segment table: logical start, K row pointer, V row pointer of each segment
    const int n_seg = a.k + 2;
    int *seg_lo = reinterpret_cast<int *>(smem_raw);                        // [n_seg+1]
    const T **seg_k = reinterpret_cast<const T **>(smem_raw + round_up((n_seg + 1) * sizeof(int), 16));
    const T **seg_v = seg_k + n_seg;
    float *red = reinterpret_cast<float *>(seg_v + n_seg);                  // [G][D+2]
    const float **seg_pos = reinterpret_cast<const float **>(red + G * (D + 2));   // [n_seg], ALiBi only
    __shared__ unsigned int s_ticket;

    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int hk = h / (a.n_heads / a.n_kv_heads);
    const int64_t row_elems = (int64_t)a.n_kv_heads * D;

    // segments: 0 = preamble, 1..k = kept paths, k+1 = tail; lengths land in seg_lo[s+1]
    for (int sgm = threadIdx.x; sgm < n_seg; sgm += kDecThreads) {
        const T *kc = static_cast<const T *>(a.k_cache) + (int64_t)hk * D;
        const T *vc = static_cast<const T *>(a.v_cache) + (int64_t)hk * D;
        int len = 0;
        int64_t row = 0;
        if (sgm == 0) {
            row = a.pre_start[b]; len = a.pre_len[b];
        } else if (sgm <= a.k) {
            const int i = a.kept_idx[(int64_t)b * a.k + sgm - 1];
            if (i >= a.ppo[b] && i < a.ppo[b + 1]) { row = a.path_start[i]; len = a.doc_len[i] + a.qry_len[i]; }
        } else {
            len = (a.tail_cap > 0 && a.tail_len) ? min(max(a.tail_len[b], 0), a.tail_cap) : 0;
            if (len) {
                kc = static_cast<const T *>(a.tail_k) + (int64_t)hk * D;
                vc = static_cast<const T *>(a.tail_v) + (int64_t)hk * D;
                row = (int64_t)b * a.tail_cap;
            }
        }
        seg_k[sgm] = kc + row * row_elems;
        seg_v[sgm] = vc + row * row_elems;
        if (ALIBI) seg_pos[sgm] = (sgm == a.k + 1 && len ? a.tail_pos : a.cache_pos) + row;
        seg_lo[sgm + 1] = len;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int cum = 0;
        seg_lo[0] = 0;
        for (int sgm = 0; sgm < n_seg; ++sgm) { cum += seg_lo[sgm + 1]; seg_lo[sgm + 1] = cum; }
    }
    __syncthreads();

    const int total = seg_lo[n_seg];
    const int chunk = (total + a.n_splits - 1) / a.n_splits;
    const int lo = min(split * chunk, total), hi = min(lo + chunk, total);

    const int g = threadIdx.x / LPK, sub = threadIdx.x % LPK;
    float qf[N];
    Vec<T>::load(static_cast<const T *>(a.q) + ((int64_t)b * a.n_heads + h) * D + sub * N, qf);
#pragma unroll
    for (int e = 0; e < N; ++e) qf[e] *= a.scale_log2e;

    float m = -INFINITY, l = 0.f, acc[N];
#pragma unroll
    for (int e = 0; e < N; ++e) acc[e] = 0.f;
    const float q_pos = ALIBI ? a.q_pos[b] : 0.f;
    const float slope_l2 = ALIBI ? a.slopes[h] * kLog2eD : 0.f;

    int seg = 0;
    for (int base = lo; base < hi; base += G * kDecUnroll) {   // trip count is block-uniform
        uint4 kr[kDecUnroll], vr[kDecUnroll];
        float kpos[kDecUnroll];
        bool live[kDecUnroll];
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {                  // all loads of the batch first
            const int j = base + g + u * G;
            live[u] = j < hi;
            if (live[u]) {
                while (j >= seg_lo[seg + 1]) ++seg;             // keys ascend: segments only advance
                const int64_t off = (int64_t)(j - seg_lo[seg]) * row_elems + sub * N;
                kr[u] = ld_stream16(seg_k[seg] + off);
                vr[u] = ld_stream16(seg_v[seg] + off);
                if (ALIBI) kpos[u] = seg_pos[seg][j - seg_lo[seg]];
            }
        }
        float s[kDecUnroll], cm = -INFINITY;
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {
            float d = 0.f;
            if (live[u]) {
                float kf[N];
                Raw16<T>::unpack(kr[u], kf);
#pragma unroll
                for (int e = 0; e < N; ++e) d = fmaf(qf[e], kf[e], d);
            }
#pragma unroll
            for (int o = LPK / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (ALIBI && live[u]) d -= slope_l2 * fabsf(q_pos - kpos[u]);
            s[u] = live[u] ? d : -INFINITY;
            cm = fmaxf(cm, s[u]);
        }
        if (cm > m) {
            const float r = ex2f(m - cm);
            l *= r;
#pragma unroll
            for (int e = 0; e < N; ++e) acc[e] *= r;
            m = cm;
        }
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {
            if (live[u]) {
                const float p = ex2f(s[u] - m);
                l += p;
                float vf[N];
                Raw16<T>::unpack(vr[u], vf);
#pragma unroll
                for (int e = 0; e < N; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
            }
        }
    }

    // ---- combine the key groups of this block (fixed order) ---------------------------
    float *mine = red + g * (D + 2);
#pragma unroll
    for (int e = 0; e < N; ++e) mine[sub * N + e] = acc[e];
    if (sub == 0) { mine[D] = m; mine[D + 1] = l; }
    __syncthreads();

    const int64_t bh = (int64_t)b * a.n_heads + h;
    float bm = -INFINITY;
    for (int i = 0; i < G; ++i) bm = fmaxf(bm, red[i * (D + 2) + D]);
    float bl = 0.f, bo = 0.f;
    if (threadIdx.x < D) {
        for (int i = 0; i < G; ++i) {
            const float gm = red[i * (D + 2) + D];
            const float w = (gm == -INFINITY) ? 0.f : ex2f(gm - bm);
            bl += red[i * (D + 2) + D + 1] * w;
            bo += red[i * (D + 2) + threadIdx.x] * w;
        }
    }

    if (a.n_splits == 1) {
        if (threadIdx.x < D) {
            const float inv = bl > 0.f ? 1.f / bl : 0.f;
            store_val(static_cast<T *>(a.out) + bh * D + threadIdx.x, bo * inv);
            if (threadIdx.x == 0 && a.lse) a.lse[bh] = bl > 0.f ? (bm + log2f(bl)) * kLn2D : -INFINITY;
        }
        return;
    }

    float *part = a.partial + (bh * a.n_splits + split) * (D + 2);
    if (threadIdx.x < D) {
        part[threadIdx.x] = bo;
        if (threadIdx.x == 0) { part[D] = bm; part[D + 1] = bl; }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_ticket = atomicAdd(a.counters + bh, 1u);
    __syncthreads();
    if (s_ticket != (unsigned)a.n_splits - 1) return;

    // last block of this (prompt, head): merge all partials in split order
    __threadfence();
    const float *all = a.partial + bh * a.n_splits * (D + 2);
    float M = -INFINITY;
    for (int i = 0; i < a.n_splits; ++i) M = fmaxf(M, __ldcg(all + i * (D + 2) + D));
    if (threadIdx.x < D) {
        float L = 0.f, O = 0.f;
        for (int i = 0; i < a.n_splits; ++i) {
            const float pm = __ldcg(all + i * (D + 2) + D);
            const float w = (pm == -INFINITY) ? 0.f : ex2f(pm - M);
            L += __ldcg(all + i * (D + 2) + D + 1) * w;
            O += __ldcg(all + i * (D + 2) + threadIdx.x) * w;
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        store_val(static_cast<T *>(a.out) + bh * D + threadIdx.x, O * inv);
        if (threadIdx.x == 0 && a.lse) a.lse[bh] = L > 0.f ? (M + log2f(L)) * kLn2D : -INFINITY;
    }
}

template <typename T, int D, bool ALIBI>
static int launch_decode_v(const DecodeArgs &a, int n_prompts, cudaStream_t st)
{
    constexpr int G = kDecThreads / (D / Vec<T>::N);
    const int n_seg = a.k + 2;
    const size_t smem = round_up((n_seg + 1) * sizeof(int), 16) + 2 * n_seg * sizeof(void *) +
                        (size_t)G * (D + 2) * sizeof(float) + (ALIBI ? n_seg * sizeof(void *) : 0);
    SP_REQUIRE(smem <= 200 * 1024, SP_ERR_UNSUPPORTED, "sp_pruned_decode: k = %d needs too much shared memory", a.k);
    if (smem > 48 * 1024)
        SP_CUDA(cudaFuncSetAttribute(decode_kernel<T, D, ALIBI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(a.n_splits, a.n_heads, n_prompts);
    decode_kernel<T, D, ALIBI><<<grid, kDecThreads, smem, st>>>(a);
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}
template <typename T, int D>
static int launch_decode(const DecodeArgs &a, int n_prompts, cudaStream_t st)
{
    return a.slopes ? launch_decode_v<T, D, true>(a, n_prompts, st) : launch_decode_v<T, D, false>(a, n_prompts, st);
}

}  // namespace sp

extern "C" size_t sp_decode_workspace_bytes(int n_prompts, int n_heads, int head_dim)
{
    using namespace sp;
    if (n_prompts <= 0 || n_heads <= 0 || head_dim <= 0) return 256;
    const size_t part = (size_t)n_prompts * n_heads * decode_split_cap(n_prompts, n_heads) *
                        (head_dim + 2) * sizeof(float);
    return 256 + decode_counter_bytes(n_prompts, n_heads) + round_up(part, 256);
}

namespace sp {
static int decode_with_workspace(const void *q, const void *k_cache, const void *v_cache,
                                 const sp_layout *lay, const int32_t *kept_idx, int k,
                                 const void *tail_k, const void *tail_v, const int32_t *tail_len,
                                 int tail_cap, int64_t max_keys, const float *q_pos, const float *cache_pos,
                                 const float *tail_pos, const float *slopes, int n_heads, int n_kv_heads,
                                 int head_dim, float scale, void *out, float *lse, void *ws,
                                 size_t ws_bytes, int dtype, void *stream)
{
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "sp_pruned_decode: unknown dtype %d", dtype);
    if (int rc = check_layout(lay)) return rc;
    SP_REQUIRE(head_dim == 64 || head_dim == 128, SP_ERR_UNSUPPORTED, "sp_pruned_decode: head_dim %d (64 or 128 supported)", head_dim);
    SP_REQUIRE(n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0, SP_ERR_INVALID_ARG,
               "sp_pruned_decode: n_heads %d must be a positive multiple of n_kv_heads %d", n_heads, n_kv_heads);
    SP_REQUIRE(k >= 0 && k <= 4096, SP_ERR_INVALID_ARG, "sp_pruned_decode: k %d out of range [0, 4096]", k);
    SP_REQUIRE(tail_cap >= 0 && max_keys >= 0, SP_ERR_INVALID_ARG, "sp_pruned_decode: negative tail_cap / max_keys");
    SP_REQUIRE(lay->n_prompts <= 65535 && n_heads <= 65535, SP_ERR_UNSUPPORTED, "sp_pruned_decode: more than 65535 prompts or heads");
    if (lay->n_prompts == 0) return SP_OK;
    SP_REQUIRE(q && out, SP_ERR_INVALID_ARG, "sp_pruned_decode: q / out is NULL");
    SP_REQUIRE(k_cache && v_cache, SP_ERR_INVALID_ARG, "sp_pruned_decode: cache pointer is NULL");
    SP_REQUIRE(k == 0 || kept_idx, SP_ERR_INVALID_ARG, "sp_pruned_decode: kept_idx is NULL with k > 0");
    SP_REQUIRE(tail_cap == 0 || (tail_k && tail_v && tail_len), SP_ERR_INVALID_ARG,
               "sp_pruned_decode: tail pointers are NULL with tail_cap > 0");
    SP_REQUIRE(aligned16(q) && aligned16(out) && aligned16(k_cache) && aligned16(v_cache) &&
                   aligned16(tail_k) && aligned16(tail_v),
               SP_ERR_INVALID_ARG, "sp_pruned_decode: data pointers must be 16-byte aligned");
    SP_REQUIRE(ws && aligned256(ws) && ws_bytes >= sp_decode_workspace_bytes(lay->n_prompts, n_heads, head_dim),
               SP_ERR_WORKSPACE, "sp_pruned_decode: workspace of %zu bytes (256-byte aligned) required",
               sp_decode_workspace_bytes(lay->n_prompts, n_heads, head_dim));

    if (max_keys == 0) max_keys = (int64_t)lay->max_pre_len + (int64_t)k * lay->max_path_len + tail_cap;
    const int cap = decode_split_cap(lay->n_prompts, n_heads);
    const int n_splits = (int)std::max<int64_t>(1, std::min<int64_t>(cap, (max_keys + 31) / 32));

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t cbytes = decode_counter_bytes(lay->n_prompts, n_heads);
    SP_CUDA(cudaMemsetAsync(ws, 0, 256 + cbytes, st));      // status word + split counters

    DecodeArgs a;
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache; a.tail_k = tail_k; a.tail_v = tail_v;
    a.ppo = lay->prompt_path_off; a.pre_start = lay->pre_start; a.pre_len = lay->pre_len;
    a.path_start = lay->path_start; a.doc_len = lay->doc_len; a.qry_len = lay->qry_len;
    a.kept_idx = kept_idx; a.tail_len = tail_len; a.out = out; a.lse = lse;
    a.counters = reinterpret_cast<unsigned int *>(static_cast<char *>(ws) + 256);
    a.partial = reinterpret_cast<float *>(static_cast<char *>(ws) + 256 + cbytes);
    a.k = k; a.tail_cap = tail_cap; a.n_heads = n_heads; a.n_kv_heads = n_kv_heads;
    a.n_splits = n_splits; a.scale_log2e = scale * kLog2eD;
    a.q_pos = q_pos; a.cache_pos = cache_pos; a.tail_pos = tail_pos; a.slopes = slopes;

    if (dtype == SP_BF16)
        return head_dim == 128 ? launch_decode<__nv_bfloat16, 128>(a, lay->n_prompts, st)
                               : launch_decode<__nv_bfloat16, 64>(a, lay->n_prompts, st);
    return head_dim == 128 ? launch_decode<float, 128>(a, lay->n_prompts, st)
                           : launch_decode<float, 64>(a, lay->n_prompts, st);
}
}  // namespace sp

extern "C" int sp_pruned_decode(const void *q, const void *k_cache, const void *v_cache,
                                const sp_layout *lay, const int32_t *kept_idx, int k,
                                const void *tail_k, const void *tail_v, const int32_t *tail_len,
                                int tail_cap, int64_t max_keys, int n_heads, int n_kv_heads,
                                int head_dim, float scale, void *out, float *lse, void *ws,
                                size_t ws_bytes, int dtype, void *stream)
{
    return sp::decode_with_workspace(q, k_cache, v_cache, lay, kept_idx, k, tail_k, tail_v, tail_len, tail_cap,
                                     max_keys, nullptr, nullptr, nullptr, nullptr, n_heads, n_kv_heads, head_dim,
                                     scale, out, lse, ws, ws_bytes, dtype, stream);
}

extern "C" int sp_pruned_decode_alibi(const void *q, const void *k_cache, const void *v_cache,
                                      const sp_layout *lay, const int32_t *kept_idx, int k,
                                      const void *tail_k, const void *tail_v, const int32_t *tail_len,
                                      int tail_cap, int64_t max_keys, const float *q_pos,
                                      const float *cache_pos, const float *tail_pos, const float *slopes,
                                      int n_heads, int n_kv_heads, int head_dim, float scale, void *out,
                                      float *lse, void *ws, size_t ws_bytes, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(lay == nullptr || lay->n_prompts == 0 || (q_pos && cache_pos && slopes && (tail_cap == 0 || tail_pos)),
               SP_ERR_INVALID_ARG, "sp_pruned_decode_alibi: q_pos, cache_pos, slopes (and tail_pos with a tail) are required");
    return decode_with_workspace(q, k_cache, v_cache, lay, kept_idx, k, tail_k, tail_v, tail_len, tail_cap, max_keys,
                                 q_pos, cache_pos, tail_pos, slopes, n_heads, n_kv_heads, head_dim, scale, out,
                                 lse, ws, ws_bytes, dtype, stream);
}

// ---------------------------------------------------------------------------------------
// sp_pruned_decode_static: the same decode kernel for callers that have no device
// allocator to ask for a workspace (see sp.h).  Its split-KV scratch (arrival counters and
// per-split partial results) lives in one fixed array inside the library image.
// ---------------------------------------------------------------------------------------
namespace sp {

constexpr size_t kStaticScratchBytes = 8u << 20;     // 8 MiB, resident on every GPU that loads the library
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static unsigned char *g_scratch_ptr[kMaxDevices] = {nullptr};   // device address of the array, per device

// In host code `g_decode_scratch` is only a handle for the runtime; the address a kernel can
// use has to be asked for, once per device, while that device is current.
static int static_scratch_address(unsigned char **out)
{
    int dev = -1;
    SP_CUDA(cudaGetDevice(&dev));
    SP_REQUIRE(dev >= 0 && dev < kMaxDevices, SP_ERR_UNSUPPORTED,
               "sp_pruned_decode_static: device ordinal %d not supported (max %d)", dev, kMaxDevices - 1);
    if (g_scratch_ptr[dev] == nullptr) {
        void *p = nullptr;
        SP_CUDA(cudaGetSymbolAddress(&p, g_decode_scratch));
        SP_REQUIRE(p != nullptr && aligned256(p), SP_ERR_CUDA,
                   "sp_pruned_decode_static: the scratch array has no usable device address");
        g_scratch_ptr[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_scratch_ptr[dev];
    return SP_OK;
}

}  // namespace sp

extern "C" size_t sp_pruned_decode_static_max_bytes(void) { return sp::kStaticScratchBytes; }

extern "C" int sp_pruned_decode_static(const void *q, const void *k_cache, const void *v_cache,
                                       const sp_layout *lay, const int32_t *kept_idx, int k,
                                       const void *tail_k, const void *tail_v,
                                       const int32_t *tail_len, int tail_cap, int64_t max_keys,
                                       int n_heads, int n_kv_heads, int head_dim, float scale,
                                       void *out, float *lse, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(dtype == SP_F32 || dtype == SP_BF16, SP_ERR_INVALID_ARG, "sp_pruned_decode_static: unknown dtype %d", dtype);
    if (int rc = check_layout(lay)) return rc;
    SP_REQUIRE(head_dim == 64 || head_dim == 128, SP_ERR_UNSUPPORTED,
               "sp_pruned_decode_static: head_dim %d (64 or 128 supported)", head_dim);
    SP_REQUIRE(n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0, SP_ERR_INVALID_ARG,
               "sp_pruned_decode_static: n_heads %d must be a positive multiple of n_kv_heads %d", n_heads, n_kv_heads);
    SP_REQUIRE(k >= 0 && k <= 4096, SP_ERR_INVALID_ARG, "sp_pruned_decode_static: k %d out of range [0, 4096]", k);
    SP_REQUIRE(tail_cap >= 0 && max_keys >= 0, SP_ERR_INVALID_ARG, "sp_pruned_decode_static: negative tail_cap / max_keys");
    SP_REQUIRE(lay->n_prompts <= 65535 && n_heads <= 65535, SP_ERR_UNSUPPORTED,
               "sp_pruned_decode_static: more than 65535 prompts or heads");
    if (lay->n_prompts == 0) return SP_OK;
    SP_REQUIRE(q && out && k_cache && v_cache, SP_ERR_INVALID_ARG, "sp_pruned_decode_static: NULL tensor");
    SP_REQUIRE(k == 0 || kept_idx, SP_ERR_INVALID_ARG, "sp_pruned_decode_static: kept_idx is NULL with k > 0");
    SP_REQUIRE(tail_cap == 0 || (tail_k && tail_v && tail_len), SP_ERR_INVALID_ARG,
               "sp_pruned_decode_static: tail pointers are NULL with tail_cap > 0");
    SP_REQUIRE(aligned16(q) && aligned16(out) && aligned16(k_cache) && aligned16(v_cache) &&
                   aligned16(tail_k) && aligned16(tail_v),
               SP_ERR_INVALID_ARG, "sp_pruned_decode_static: data pointers must be 16-byte aligned");

    if (max_keys == 0) max_keys = (int64_t)lay->max_pre_len + (int64_t)k * lay->max_path_len + tail_cap;
    const int cap = decode_split_cap(lay->n_prompts, n_heads);
    const int n_splits = (int)std::max<int64_t>(1, std::min<int64_t>(cap, (max_keys + 31) / 32));
    const size_t cbytes = decode_counter_bytes(lay->n_prompts, n_heads);
    const size_t pbytes = n_splits > 1
        ? (size_t)lay->n_prompts * n_heads * n_splits * (head_dim + 2) * sizeof(float) : 0;
    SP_REQUIRE(cbytes + pbytes <= kStaticScratchBytes, SP_ERR_WORKSPACE,
               "sp_pruned_decode_static: this problem needs %zu bytes of split-KV scratch but the built-in "
               "array holds %zu; use sp_pruned_decode with a caller workspace",
               cbytes + pbytes, kStaticScratchBytes);

    unsigned char *scratch = nullptr;
    if (int rc = static_scratch_address(&scratch)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array still holds the previous call's counters: they must start at zero
    SP_CUDA(cudaMemsetAsync(scratch, 0, cbytes, st));

    DecodeArgs a;
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache; a.tail_k = tail_k; a.tail_v = tail_v;
    a.ppo = lay->prompt_path_off; a.pre_start = lay->pre_start; a.pre_len = lay->pre_len;
    a.path_start = lay->path_start; a.doc_len = lay->doc_len; a.qry_len = lay->qry_len;
    a.kept_idx = kept_idx; a.tail_len = tail_len; a.out = out; a.lse = lse;
    a.counters = reinterpret_cast<unsigned int *>(scratch);
    a.partial = reinterpret_cast<float *>(scratch + cbytes);
    a.k = k; a.tail_cap = tail_cap; a.n_heads = n_heads; a.n_kv_heads = n_kv_heads;
    a.n_splits = n_splits; a.scale_log2e = scale * kLog2eD;
    a.q_pos = nullptr; a.cache_pos = nullptr; a.tail_pos = nullptr; a.slopes = nullptr;

    if (dtype == SP_BF16)
        return head_dim == 128 ? launch_decode<__nv_bfloat16, 128>(a, lay->n_prompts, st)
                               : launch_decode<__nv_bfloat16, 64>(a, lay->n_prompts, st);
    return head_dim == 128 ? launch_decode<float, 128>(a, lay->n_prompts, st)
                           : launch_decode<float, 64>(a, lay->n_prompts, st);
}
