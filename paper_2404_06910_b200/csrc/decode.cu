// sp_pruned_decode: one-token decode attention over the pruned cache (Section 3.2.3;
// Algorithm 3: preamble + kept (document + query) + task/response tokens).
//
// HBM-bound: every kept K and V row is read exactly once.  Pruning is an index list --
// the kernel walks [preamble | kept path ranges | tail] as one logical key sequence and
// never copies KV.  The sequence is split across blocks (split-KV) so that small batches
// still fill the machine; each block keeps an online softmax per key group, writes one
// partial (max, sum, unnormalised output), and the last block to finish a (prompt, head)
// merges the partials in split order, so results do not depend on scheduling.
#include <cooperative_groups.h>

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
    int64_t total_tokens;    // T: cache segments outside [0, T) are skipped (cluster kernel)
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
    const int64_t want = (8LL * num_sms()) / bh;      // 8 blocks per SM: all blocks of a launch are resident at once
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


// ---------------------------------------------------------------------------------------
// Cluster variant (the one sp_pruned_decode runs): the blocks that split one (prompt, KV head)
// form a thread-block cluster and merge their partial results through distributed shared
// memory, in split order.  No global scratch, no counters to clear, no atomics.  A block owns
// a KV head and GRP of its query heads, so grouped heads read every K and V row once.
// ROPE: the query rows and the newest tail key arrive unrotated and are rotated here, at the
// new token's real-valued position (Section 3.2.2), which saves the separate launch a decode
// step otherwise needs; the rotated key is written back to the tail for the later steps.
// ---------------------------------------------------------------------------------------
struct DecodeRope {
    double inv_freq[64];      // base^(-2m/D), m < D/2 <= 64
};

// MINB: resident blocks per SM the register budget is sized for.  Split launches want 8 (a whole
// launch in one wave, clusters of 2^n blocks pack evenly); an unsplit launch over a large batch
// runs faster with the few registers more that 7 leave (nothing spills).
template <typename T, int D, int GRP, bool ALIBI, bool ROPE, int MINB>
__global__ void __launch_bounds__(kDecThreads, MINB)
decode_cluster_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ DecodeRope rope, int rope_pairing)
{
    namespace cg = cooperative_groups;
    constexpr int N = Vec<T>::N;            // elements per 16-byte load
    constexpr int LPK = D / N;              // lanes that share one key row
    constexpr int G = kDecThreads / LPK;    // key groups per block
    constexpr int PS = D + 2;               // one partial: D outputs, max, sum
    static_assert(LPK <= 32 && (32 % LPK) == 0, "a key row must fit in one warp");

    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int n_seg = a.k + 2;
    int *seg_lo = reinterpret_cast<int *>(smem_raw);                        // [n_seg+1]
    const T **seg_k = reinterpret_cast<const T **>(smem_raw + round_up((n_seg + 1) * sizeof(int), 16));
    const T **seg_v = seg_k + n_seg;
    const float **seg_pos = reinterpret_cast<const float **>(seg_v + n_seg);       // [n_seg], ALiBi only
    float *red = reinterpret_cast<float *>(seg_pos + n_seg);                // [G][GRP][PS]
    float *part = red + G * GRP * PS;                                       // [GRP][PS], read by the cluster's first block
    float2 *cs = reinterpret_cast<float2 *>(part + GRP * PS);               // [D/2] (cos, sin), ROPE only

    const int split = blockIdx.x, b = blockIdx.z;
    const int group = a.n_heads / a.n_kv_heads;                 // query heads per KV head
    const int per_kv = group / GRP;                             // blocks (in y) per KV head
    const int hk = blockIdx.y / per_kv;
    const int h0 = hk * group + (blockIdx.y - hk * per_kv) * GRP;   // first query head of this block
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
        // a cache segment that the device-side layout puts outside the tensors is not read at all
        if (sgm <= a.k && (len < 0 || row < 0 || row + len > a.total_tokens)) { len = 0; row = 0; }
        seg_k[sgm] = kc + row * row_elems;
        seg_v[sgm] = vc + row * row_elems;
        if (ALIBI) seg_pos[sgm] = (sgm == a.k + 1 && len ? a.tail_pos : a.cache_pos) + row;
        seg_lo[sgm + 1] = len;
    }
    if (ROPE && threadIdx.x < D / 2) {
        // The angle is formed in fp64 at the real-valued position and brought into [-pi, pi] there
        // (two fused steps with a split 2 pi); the small remainder goes through the fp32 sine and
        // cosine, whose error is then far below one rounding of the rotated values.
        const double ang = (double)a.q_pos[b] * rope.inv_freq[threadIdx.x];
        const double turns = rint(ang * 0.15915494309189535);
        const double r = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, ang));
        float sn, cn;
        sincosf((float)r, &sn, &cn);
        cs[threadIdx.x] = make_float2(cn, sn);
    }
    __syncthreads();
    if (threadIdx.x < 32) {                 // prefix sum of the lengths, 32 segments per round
        int carry = 0;
        if (threadIdx.x == 0) seg_lo[0] = 0;
        for (int base = 0; base < n_seg; base += 32) {
            const int sgm = base + (int)threadIdx.x;
            int v = sgm < n_seg ? seg_lo[sgm + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, v, o);
                if ((int)threadIdx.x >= o) v += up;
            }
            if (sgm < n_seg) seg_lo[sgm + 1] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();

    const int total = seg_lo[n_seg];
    const int chunk = (total + a.n_splits - 1) / a.n_splits;
    const int lo = min(split * chunk, total), hi = min(lo + chunk, total);
    // ROPE: the newest tail row (the last key of the sequence, when there is a tail) is still unrotated
    const int j_new = (ROPE && seg_lo[n_seg] > seg_lo[n_seg - 1]) ? total - 1 : -1;
    const bool owns_new = j_new >= lo && j_new < hi;                 // block-uniform; j_new is then hi - 1
    const int hi_loop = owns_new ? hi - 1 : hi;                        // the new key is handled after the loop

    const int g = threadIdx.x / LPK, sub = threadIdx.x % LPK;
    // rotates the N elements this lane holds of a D-vector spread over LPK lanes
    auto rotate = [&](float (&f)[N]) {
        if (rope_pairing == SP_ROPE_HALF_SPLIT) {
            const bool upper = sub >= LPK / 2;
            const int m0 = (upper ? sub - LPK / 2 : sub) * N;
#pragma unroll
            for (int e = 0; e < N; ++e) {
                const float other = __shfl_xor_sync(0xffffffffu, f[e], LPK / 2);
                const float2 w = cs[m0 + e];
                f[e] = upper ? fmaf(other, w.y, f[e] * w.x) : fmaf(-other, w.y, f[e] * w.x);
            }
        } else {
#pragma unroll
            for (int e = 0; e < N; e += 2) {
                const float2 w = cs[(sub * N + e) >> 1];
                const float x0 = f[e], x1 = f[e + 1];
                f[e] = x0 * w.x - x1 * w.y;
                f[e + 1] = x0 * w.y + x1 * w.x;
            }
        }
    };

    float qf[GRP][N];
#pragma unroll
    for (int r = 0; r < GRP; ++r) {
        Vec<T>::load(static_cast<const T *>(a.q) + ((int64_t)b * a.n_heads + h0 + r) * D + sub * N, qf[r]);
        if (ROPE) {
            rotate(qf[r]);
#pragma unroll
            for (int e = 0; e < N; ++e) qf[r][e] = to_float(T(qf[r][e]));   // the rounding a stored rotated query has
        }
#pragma unroll
        for (int e = 0; e < N; ++e) qf[r][e] *= a.scale_log2e;
    }

    float m[GRP], l[GRP], acc[GRP][N];
#pragma unroll
    for (int r = 0; r < GRP; ++r) {
        m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
        for (int e = 0; e < N; ++e) acc[r][e] = 0.f;
    }
    const float q_pos = ALIBI ? a.q_pos[b] : 0.f;
    float slope_l2[GRP];
#pragma unroll
    for (int r = 0; r < GRP; ++r) slope_l2[r] = ALIBI ? a.slopes[h0 + r] * kLog2eD : 0.f;

    int seg = 0;
    for (int base = lo; base < hi_loop; base += G * kDecUnroll) {   // trip count is block-uniform
        uint4 kr[kDecUnroll], vr[kDecUnroll];
        float kpos[kDecUnroll];
        bool live[kDecUnroll];
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {                  // all loads of the batch first
            const int j = base + g + u * G;
            live[u] = j < hi_loop;
            if (live[u]) {
                while (j >= seg_lo[seg + 1]) ++seg;             // keys ascend: segments only advance
                const int64_t off = (int64_t)(j - seg_lo[seg]) * row_elems + sub * N;
                kr[u] = ld_stream16(seg_k[seg] + off);
                vr[u] = ld_stream16(seg_v[seg] + off);
                if (ALIBI) kpos[u] = seg_pos[seg][j - seg_lo[seg]];
            }
        }
        float s[GRP][kDecUnroll], cm[GRP];
#pragma unroll
        for (int r = 0; r < GRP; ++r) cm[r] = -INFINITY;
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {
            float kf[N];
            if (live[u]) Raw16<T>::unpack(kr[u], kf);
#pragma unroll
            for (int r = 0; r < GRP; ++r) {
                float d = 0.f;
                if (live[u]) {
#pragma unroll
                    for (int e = 0; e < N; ++e) d = fmaf(qf[r][e], kf[e], d);
                }
#pragma unroll
                for (int o = LPK / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if (ALIBI && live[u]) d -= slope_l2[r] * fabsf(q_pos - kpos[u]);
                s[r][u] = live[u] ? d : -INFINITY;
                cm[r] = fmaxf(cm[r], s[r][u]);
            }
        }
#pragma unroll
        for (int r = 0; r < GRP; ++r) {
            if (cm[r] > m[r]) {
                const float sc = ex2f(m[r] - cm[r]);
                l[r] *= sc;
#pragma unroll
                for (int e = 0; e < N; ++e) acc[r][e] *= sc;
                m[r] = cm[r];
            }
        }
#pragma unroll
        for (int u = 0; u < kDecUnroll; ++u) {
            if (live[u]) {
                float vf[N];
                Raw16<T>::unpack(vr[u], vf);
#pragma unroll
                for (int r = 0; r < GRP; ++r) {
                    const float p = ex2f(s[r][u] - m[r]);
                    l[r] += p;
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[r][e] = fmaf(p, vf[e], acc[r][e]);
                }
            }
        }
    }

    if (ROPE && owns_new && threadIdx.x < 32) {
        // The newest key, outside the streaming loop: warp 0 loads the unrotated row (every key
        // group of the warp holds a copy), rotates it, group 0 writes it back for the later steps
        // and takes it into its running softmax like any other key.
        const int64_t off = (int64_t)(j_new - seg_lo[n_seg - 1]) * row_elems + sub * N;
        T *krow = const_cast<T *>(seg_k[n_seg - 1]) + off;
        float kf[N], vf[N];
        Vec<T>::load(krow, kf);
        Vec<T>::load(seg_v[n_seg - 1] + off, vf);
        rotate(kf);
#pragma unroll
        for (int e = 0; e < N; ++e) kf[e] = to_float(T(kf[e]));           // as it is stored
        if (g == 0) {
#pragma unroll
            for (int e = 0; e < N; ++e) store_val(krow + e, kf[e]);
        }
#pragma unroll
        for (int r = 0; r < GRP; ++r) {
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < N; ++e) d = fmaf(qf[r][e], kf[e], d);
#pragma unroll
            for (int o = LPK / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
            if (g == 0) {
                if (d > m[r]) {
                    const float sc = ex2f(m[r] - d);
                    l[r] *= sc;
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[r][e] *= sc;
                    m[r] = d;
                }
                const float p = ex2f(d - m[r]);
                l[r] += p;
#pragma unroll
                for (int e = 0; e < N; ++e) acc[r][e] = fmaf(p, vf[e], acc[r][e]);
            }
        }
    }

    // ---- combine the key groups of this block (fixed order) ---------------------------
#pragma unroll
    for (int r = 0; r < GRP; ++r) {
        float *mine = red + (g * GRP + r) * PS;
#pragma unroll
        for (int e = 0; e < N; ++e) mine[sub * N + e] = acc[r][e];
        if (sub == 0) { mine[D] = m[r]; mine[D + 1] = l[r]; }
    }
    __syncthreads();

    float bm[GRP], bl[GRP], bo[GRP];
#pragma unroll
    for (int r = 0; r < GRP; ++r) {
        bm[r] = -INFINITY; bl[r] = 0.f; bo[r] = 0.f;
        for (int i = 0; i < G; ++i) bm[r] = fmaxf(bm[r], red[(i * GRP + r) * PS + D]);
        if (threadIdx.x < D) {
            for (int i = 0; i < G; ++i) {
                const float gm = red[(i * GRP + r) * PS + D];
                const float w = (gm == -INFINITY) ? 0.f : ex2f(gm - bm[r]);
                bl[r] += red[(i * GRP + r) * PS + D + 1] * w;
                bo[r] += red[(i * GRP + r) * PS + threadIdx.x] * w;
            }
        }
    }

    if (a.n_splits > 1) {
        // ---- merge the splits through the cluster's shared memory, in split order ---------
        cg::cluster_group cluster = cg::this_cluster();
        if (threadIdx.x < D) {
#pragma unroll
            for (int r = 0; r < GRP; ++r) {
                part[r * PS + threadIdx.x] = bo[r];
                if (threadIdx.x == 0) { part[r * PS + D] = bm[r]; part[r * PS + D + 1] = bl[r]; }
            }
        }
        cluster.sync();
        if (split == 0 && threadIdx.x < D) {
#pragma unroll
            for (int r = 0; r < GRP; ++r) {
                float M = -INFINITY;
                for (int i = 0; i < a.n_splits; ++i) M = fmaxf(M, cluster.map_shared_rank(part, i)[r * PS + D]);
                float L = 0.f, O = 0.f;
                for (int i = 0; i < a.n_splits; ++i) {
                    const float *rp = cluster.map_shared_rank(part, i) + r * PS;
                    const float w = (rp[D] == -INFINITY) ? 0.f : ex2f(rp[D] - M);
                    L += rp[D + 1] * w;
                    O += rp[threadIdx.x] * w;
                }
                bm[r] = M; bl[r] = L; bo[r] = O;
            }
        }
        cluster.sync();                     // the others' shared memory stays alive until it has been read
        if (split != 0) return;
    }
    if (threadIdx.x < D) {
#pragma unroll
        for (int r = 0; r < GRP; ++r) {
            const int64_t bh = (int64_t)b * a.n_heads + h0 + r;
            const float inv = bl[r] > 0.f ? 1.f / bl[r] : 0.f;
            store_val(static_cast<T *>(a.out) + bh * D + threadIdx.x, bo[r] * inv);
            if (threadIdx.x == 0 && a.lse) a.lse[bh] = bl[r] > 0.f ? (bm[r] + log2f(bl[r])) * kLn2D : -INFINITY;
        }
    }
}

// Splits of a launch: a power of two (cluster size), at most 16, such that one launch stays
// within about one resident wave and a split keeps at least 32 keys.
static int cluster_splits(int n_prompts, int blocks_y, int64_t max_keys, int blocks_per_sm)
{
    const int64_t by = std::max<int64_t>(1, (int64_t)n_prompts * blocks_y);
    const int64_t want = std::min<int64_t>(((int64_t)blocks_per_sm * num_sms()) / by, (max_keys + 31) / 32);
    int n = 1;
    while (n * 2 <= want && n < 16) n *= 2;
    return n;
}

template <typename T, int D, int GRP, bool ALIBI, bool ROPE>
static int launch_decode_cluster(DecodeArgs a, const DecodeRope &rope, int pairing, int n_prompts, int64_t max_keys,
                                 cudaStream_t st)
{
    constexpr int G = kDecThreads / (D / Vec<T>::N);
    constexpr int PS = D + 2;
    const int group = a.n_heads / a.n_kv_heads;
    const int blocks_y = a.n_kv_heads * (group / GRP);
    constexpr int kMinB = GRP == 1 ? 8 : (GRP == 2 ? 5 : 3);
    a.n_splits = cluster_splits(n_prompts, blocks_y, max_keys, kMinB);
    const int n_seg = a.k + 2;
    const size_t smem = round_up((n_seg + 1) * sizeof(int), 16) + 3 * n_seg * sizeof(void *) +
                        (size_t)(G + 1) * GRP * PS * sizeof(float) + (D / 2) * sizeof(float2);
    SP_REQUIRE(smem <= 200 * 1024, SP_ERR_UNSUPPORTED, "sp_pruned_decode: k = %d needs too much shared memory", a.k);
    auto kern = (GRP == 1 && a.n_splits == 1) ? decode_cluster_kernel<T, D, GRP, ALIBI, ROPE, kMinB - (GRP == 1 ? 1 : 0)>
                                              : decode_cluster_kernel<T, D, GRP, ALIBI, ROPE, kMinB>;
    if (smem > 48 * 1024)
        SP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (a.n_splits > 8)
        SP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.n_splits, blocks_y, n_prompts);
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = a.n_splits; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.n_splits > 1 ? 1 : 0;      // one block per (prompt, KV head group): a plain launch
    SP_CUDA(cudaLaunchKernelEx(&cfg, kern, a, rope, pairing));
    return SP_OK;
}

template <typename T, int D, bool ALIBI, bool ROPE>
static int launch_decode_grp(const DecodeArgs &a, const DecodeRope &rope, int pairing, int n_prompts, int64_t max_keys,
                             cudaStream_t st)
{
    // query heads per block: the largest of 4, 2, 1 that divides the group, so grouped heads share
    // one pass over their K and V rows
    const int group = a.n_heads / a.n_kv_heads;
    if (group % 4 == 0) return launch_decode_cluster<T, D, 4, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st);
    if (group % 2 == 0) return launch_decode_cluster<T, D, 2, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st);
    return launch_decode_cluster<T, D, 1, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st);
}

template <bool ALIBI, bool ROPE>
static int launch_decode_any(const DecodeArgs &a, const DecodeRope &rope, int pairing, int n_prompts, int64_t max_keys,
                             int head_dim, int dtype, cudaStream_t st)
{
    if (dtype == SP_BF16)
        return head_dim == 128 ? launch_decode_grp<__nv_bfloat16, 128, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st)
                               : launch_decode_grp<__nv_bfloat16, 64, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st);
    return head_dim == 128 ? launch_decode_grp<float, 128, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st)
                           : launch_decode_grp<float, 64, ALIBI, ROPE>(a, rope, pairing, n_prompts, max_keys, st);
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
                                 const float *tail_pos, const float *slopes, double rope_base, int pairing,
                                 int n_heads, int n_kv_heads, int head_dim, float scale, void *out, float *lse,
                                 void *ws, size_t ws_bytes, bool ws_required, int dtype, void *stream)
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
    if (ws_required)
        SP_REQUIRE(ws && aligned256(ws) && ws_bytes >= sp_decode_workspace_bytes(lay->n_prompts, n_heads, head_dim),
                   SP_ERR_WORKSPACE, "sp_pruned_decode: workspace of %zu bytes (256-byte aligned) required",
                   sp_decode_workspace_bytes(lay->n_prompts, n_heads, head_dim));

    if (max_keys == 0) max_keys = (int64_t)lay->max_pre_len + (int64_t)k * lay->max_path_len + tail_cap;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // The cluster kernel needs no scratch: the workspace is accepted (and checked) for the sake of
    // the interface, and its status word is left alone (this call has no bounded waits).
    DecodeArgs a;
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache; a.tail_k = tail_k; a.tail_v = tail_v;
    a.ppo = lay->prompt_path_off; a.pre_start = lay->pre_start; a.pre_len = lay->pre_len;
    a.path_start = lay->path_start; a.doc_len = lay->doc_len; a.qry_len = lay->qry_len;
    a.kept_idx = kept_idx; a.tail_len = tail_len; a.out = out; a.lse = lse;
    a.counters = nullptr; a.partial = nullptr;
    a.k = k; a.tail_cap = tail_cap; a.n_heads = n_heads; a.n_kv_heads = n_kv_heads;
    a.n_splits = 1; a.scale_log2e = scale * kLog2eD; a.total_tokens = lay->total_tokens;
    a.q_pos = q_pos; a.cache_pos = cache_pos; a.tail_pos = tail_pos; a.slopes = slopes;

    DecodeRope rope = {};
    if (rope_base > 0.0) {
        SP_REQUIRE(slopes == nullptr, SP_ERR_INVALID_ARG, "sp_pruned_decode: rotary and ALiBi variants exclude each other");
        const int group = n_heads / n_kv_heads;
        SP_REQUIRE(group == 1 || group == 2 || group == 4, SP_ERR_UNSUPPORTED,
                   "sp_pruned_decode_rope: %d query heads per KV head (1, 2 or 4 supported: one block must own the new key)", group);
        for (int m = 0; m < head_dim / 2; ++m) rope.inv_freq[m] = std::pow(rope_base, -2.0 * m / head_dim);
        return launch_decode_any<false, true>(a, rope, pairing, lay->n_prompts, max_keys, head_dim, dtype, st);
    }
    return slopes ? launch_decode_any<true, false>(a, rope, 0, lay->n_prompts, max_keys, head_dim, dtype, st)
                  : launch_decode_any<false, false>(a, rope, 0, lay->n_prompts, max_keys, head_dim, dtype, st);
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
                                     max_keys, nullptr, nullptr, nullptr, nullptr, 0.0, 0, n_heads, n_kv_heads, head_dim,
                                     scale, out, lse, ws, ws_bytes, true, dtype, stream);
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
                                 q_pos, cache_pos, tail_pos, slopes, 0.0, 0, n_heads, n_kv_heads, head_dim, scale, out,
                                 lse, ws, ws_bytes, true, dtype, stream);
}

extern "C" int sp_pruned_decode_rope(const void *q, const void *k_cache, const void *v_cache,
                                     const sp_layout *lay, const int32_t *kept_idx, int k, void *tail_k,
                                     const void *tail_v, const int32_t *tail_len, int tail_cap, int64_t max_keys,
                                     const float *q_pos, double rope_base, int pairing, int n_heads, int n_kv_heads,
                                     int head_dim, float scale, void *out, float *lse, int dtype, void *stream)
{
    using namespace sp;
    SP_REQUIRE(rope_base > 0.0, SP_ERR_INVALID_ARG, "sp_pruned_decode_rope: base must be positive");
    SP_REQUIRE(pairing == SP_ROPE_HALF_SPLIT || pairing == SP_ROPE_INTERLEAVED, SP_ERR_INVALID_ARG,
               "sp_pruned_decode_rope: unknown pairing %d", pairing);
    SP_REQUIRE(lay == nullptr || lay->n_prompts == 0 || q_pos, SP_ERR_INVALID_ARG, "sp_pruned_decode_rope: q_pos is NULL");
    return decode_with_workspace(q, k_cache, v_cache, lay, kept_idx, k, tail_k, tail_v, tail_len, tail_cap, max_keys,
                                 q_pos, nullptr, nullptr, nullptr, rope_base, pairing, n_heads, n_kv_heads, head_dim,
                                 scale, out, lse, nullptr, 0, false, dtype, stream);
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
    a.n_splits = n_splits; a.scale_log2e = scale * kLog2eD; a.total_tokens = lay->total_tokens;
    a.q_pos = nullptr; a.cache_pos = nullptr; a.tail_pos = nullptr; a.slopes = nullptr;

    if (dtype == SP_BF16)
        return head_dim == 128 ? launch_decode<__nv_bfloat16, 128>(a, lay->n_prompts, st)
                               : launch_decode<__nv_bfloat16, 64>(a, lay->n_prompts, st);
    return head_dim == 128 ? launch_decode<float, 128>(a, lay->n_prompts, st)
                           : launch_decode<float, 64>(a, lay->n_prompts, st);
}
