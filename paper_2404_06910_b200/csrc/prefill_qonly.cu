// Query rows only: the N query copies of a prompt attend to cached preamble and document
// keys and, causally, to their own rows (Section 3.3, path caching: at serving time only the
// query segments are new).  bf16, head_dim 128.
//
// With 24-32 query rows per path the work is a stream over the cached K/V with ~25 flop per
// byte, so the kernel is built for HBM: work item = (32 query rows, head); two warps of 16
// rows each; keys arrive 32 at a time through a three-stage cp.async ring that runs on across
// item boundaries (the next item's first tiles and its Q are in flight while the current item
// finishes); S = Q K^T and O += P V with warp-level mma.sync m16n8k16 from 16-byte-swizzled
// shared memory (ldmatrix), online softmax in registers.  128 query rows would fill a
// tcgen05 tile, 32 rows fill a quarter of one, and the tensor pipe is idle either way at this
// intensity; small warp-level tiles keep many independent items in flight per SM instead.
// The grid is persistent with the head as the fastest index, like the full prefill.
#include "common.cuh"
#include "prefill_plan.cuh"

namespace sp {

constexpr int kQM = 32;               // query rows per item
constexpr int kQN = 32;               // keys per tile
constexpr int kQD = 128;              // head_dim
constexpr int kQStages = 3;
constexpr int kQThreads = 64;         // two warps x 16 query rows
constexpr int kQBlocksPerSM = 4;
constexpr int kRowB = kQD * 2;        // bytes of one (token, head) row
constexpr int kTileB = kQN * kRowB;   // 8 KB: one K or V tile, also one Q tile
constexpr float kLog2eQ = 1.4426950408889634f;
constexpr float kLn2Q = 0.6931471805599453f;

struct QoParams {
    const unsigned char *q, *k, *v;
    unsigned char *out;
    float *lse;
    const TcHeader *hdr;
    const TcTile *tiles;
    int n_heads, n_kv_heads, kv_group;
    int64_t total_tokens;
    float scale_log2e;
    const float *pos, *slopes;       // ALiBi variant: token positions [T], head slopes [H]
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte piece `chunk` of row `row` of a [rows][256 B] tile; pieces are xor-swizzled by the
// row so that the eight rows an ldmatrix touches fall into different banks.
__device__ __forceinline__ uint32_t sw_off(int row, int chunk) { return (uint32_t)(row * kRowB + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 16 : 0;     // 0: the 16 bytes are zero-filled, the source is not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2q(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

struct QKv {
    int row0;        // packed row of the tile's first key
    int n_valid;     // keys that exist (1..kQN)
    int k_off;       // own-segment offset of the first key; -1 for preamble tiles
};

// Walks the block's items (query tile, head) in grid-stride order and, inside an item, its
// key tiles: the preamble's, then the segment's own up to the tile's last query row.
// g counts key tiles since the block started and selects the ring stage.
struct QCursor {
    const TcTile *tiles;
    uint32_t it, n_items, stride, g, item_no;
    int n_heads, h, j, n_kv, n_pre;
    TcTile t;
    bool valid;
    __device__ __forceinline__ void load()
    {
        valid = it < n_items;
        if (valid) {
            const uint32_t ti = it / (uint32_t)n_heads;
            h = (int)(it - ti * (uint32_t)n_heads);
            t = tiles[ti];
            n_pre = (t.pre_len + kQN - 1) / kQN;
            n_kv = n_pre + (t.q_off + t.n_rows + kQN - 1) / kQN;
            j = 0;
        }
    }
    __device__ __forceinline__ void init(const TcTile *tl, uint32_t n, int heads)
    {
        tiles = tl; n_items = n; n_heads = heads; it = blockIdx.x; stride = gridDim.x; g = 0; item_no = 0;
        load();
    }
    __device__ __forceinline__ QKv kv() const
    {
        QKv k;
        if (j < n_pre) {
            k.row0 = t.pre_row + j * kQN; k.n_valid = min(kQN, t.pre_len - j * kQN); k.k_off = -1;
        } else {
            const int o = (j - n_pre) * kQN;
            k.row0 = t.own_row + o; k.n_valid = min(kQN, t.q_off + t.n_rows - o); k.k_off = o;
        }
        return k;
    }
    __device__ __forceinline__ void next()
    {
        ++g;
        if (++j == n_kv) { it += stride; ++item_no; load(); }
    }
    __device__ __forceinline__ bool last_of_item() const { return j == n_kv - 1; }
};

// Copies n_valid rows (of one head) into a swizzled [32][256 B] tile; the rest is zero-filled.
__device__ __forceinline__ void load_rows(unsigned char *dst, const unsigned char *src, int64_t pitch, int row0, int n_valid)
{
    const uint32_t d = smem_addr(dst);
#pragma unroll
    for (int i = 0; i < kQN * 16 / kQThreads; ++i) {
        const int idx = (int)threadIdx.x + kQThreads * i, row = idx >> 4, chunk = idx & 15;
        const bool ok = row < n_valid;
        cp_async16(d + sw_off(row, chunk), src + (int64_t)(row0 + (ok ? row : 0)) * pitch + chunk * 16, ok);
    }
}

// ALIBI: scores get -slope_h * |pos_q - pos_k| before the softmax (Section 3.2.2).
template <bool ALIBI>
__global__ void __launch_bounds__(kQThreads, kQBlocksPerSM) prefill_qonly_kernel(const QoParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sK = smem;                               // [stages] 32 keys x 256 B
    unsigned char *sV = sK + kQStages * kTileB;             // [stages]
    unsigned char *sQ = sV + kQStages * kTileB;             // one item's 32 query rows

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const uint32_t n_items = p.hdr->n_tiles * (uint32_t)p.n_heads;
    const int64_t q_pitch = (int64_t)p.n_heads * kRowB, kv_pitch = (int64_t)p.n_kv_heads * kRowB;

    QCursor lc, cc;                  // lc: next tile to fetch; cc: next tile to compute
    lc.init(p.tiles, n_items, p.n_heads);
    cc = lc;

    // Fetches run up to kQStages - 1 tiles ahead of the arithmetic, one cp.async group per tile.
    // A new item's Q may replace the previous one only once both warps hold that one in
    // registers (q_held: the last item whose Q fragments were loaded); until then the fetch
    // cursor waits, which only happens behind items of one or two key tiles.
    int q_held = -1;
    auto fetch_one = [&]() {
        const int st = lc.g % kQStages;
        const QKv kt = lc.kv();
        const int64_t col = (int64_t)(lc.h / p.kv_group) * kRowB;
        if (lc.j == 0)
            load_rows(sQ, p.q + (int64_t)lc.h * kRowB, q_pitch, lc.t.q_row, lc.t.n_rows);
        load_rows(sK + st * kTileB, p.k + col, kv_pitch, kt.row0, kt.n_valid);
        load_rows(sV + st * kTileB, p.v + col, kv_pitch, kt.row0, kt.n_valid);
        cp_async_commit();
        lc.next();
    };
    auto q_slot_busy = [&]() { return lc.j == 0 && (int)lc.item_no > q_held + 1; };
    // prologue: one tile fewer than later on, no stage has been consumed yet
    while (lc.valid && lc.g < kQStages - 1 && !q_slot_busy()) fetch_one();

    uint32_t qf[kQD / 16][4];        // this warp's 16 query rows as A fragments
    float o[kQD / 8][4];             // O accumulator: 16 rows x 128 columns
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // rows gid and gid + 8
    float pq[2] = {0.f, 0.f}, slope_l2 = 0.f;                         // ALiBi: the two rows' positions

    while (cc.valid) {
        // tile cc.g must have landed: all groups but the ones of the tiles fetched after it
        const int pend = (int)(lc.g - cc.g) - 1;
        if (pend >= 2) cp_async_wait<2>(); else if (pend == 1) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncthreads();             // ... for every thread; and the stage of tile cc.g - 1 is free
        if (cc.j == 0) {
            const uint32_t qb = smem_addr(sQ);
#pragma unroll
            for (int ks = 0; ks < kQD / 16; ++ks)
                ldsm_x4(qb + sw_off(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, ks * 2 + (lane >> 4)), qf[ks]);
#pragma unroll
            for (int i = 0; i < kQD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
            m_run[0] = m_run[1] = -INFINITY; l_run[0] = l_run[1] = 0.f;
            if (ALIBI) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int rowq = warp * 16 + gid + 8 * hh;
                    pq[hh] = rowq < cc.t.n_rows ? p.pos[cc.t.q_row + rowq] : 0.f;
                }
                slope_l2 = p.slopes[cc.h] * kLog2eQ;
            }
            __syncthreads();         // both warps hold their Q before the next item's may be fetched
            q_held = (int)cc.item_no;
        }
        while (lc.valid && lc.g < cc.g + kQStages && !q_slot_busy()) fetch_one();

        const int st = cc.g % kQStages;
        const QKv kt = cc.kv();
        const uint32_t kb = smem_addr(sK + st * kTileB), vb = smem_addr(sV + st * kTileB);

        // ---- S = Q K^T: 16 rows x 32 keys
        float s[kQN / 8][4];
#pragma unroll
        for (int i = 0; i < kQN / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kQD / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < kQN / 16; ++np) {
                uint32_t b[4];
                ldsm_x4(kb + sw_off(np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8, ks * 2 + ((lane >> 3) & 1)), b);
                mma_bf16(s[2 * np], qf[ks], b[0], b[1]);
                mma_bf16(s[2 * np + 1], qf[ks], b[2], b[3]);
            }
        }

        // ---- online softmax (log2 units); keys past a row's limit count as -inf
        uint32_t pa[kQN / 16][4];
        float pk[kQN / 8][2];        // ALiBi: positions of this thread's eight key columns
        if (ALIBI) {
#pragma unroll
            for (int nt = 0; nt < kQN / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int col = nt * 8 + 2 * tig + e;
                    pk[nt][e] = col < kt.n_valid ? p.pos[kt.row0 + col] : 0.f;
                }
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int rowq = warp * 16 + gid + 8 * hh;
            const int lim = kt.k_off < 0 ? kt.n_valid : min(kt.n_valid, cc.t.q_off + rowq - kt.k_off + 1);
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < kQN / 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int col = nt * 8 + 2 * tig + e;
                    float x = s[nt][2 * hh + e] * p.scale_log2e;
                    if (ALIBI) x -= slope_l2 * fabsf(pq[hh] - pk[nt][e]);
                    x = col < lim ? x : -INFINITY;
                    s[nt][2 * hh + e] = x;
                    mx = fmaxf(mx, x);
                }
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[hh], mx);
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = ex2q(m_run[hh] - m_use);
            m_run[hh] = m_new;
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < kQN / 8; ++nt) {
                const float p0 = ex2q(s[nt][2 * hh] - m_use), p1 = ex2q(s[nt][2 * hh + 1] - m_use);
                sum += p0 + p1;
                pa[nt >> 1][(nt & 1) * 2 + hh] = pack2(p0, p1);
            }
            l_run[hh] = l_run[hh] * alpha + sum;     // per-thread partial; the quad is summed at the end
#pragma unroll
            for (int i = 0; i < kQD / 8; ++i) { o[i][2 * hh] *= alpha; o[i][2 * hh + 1] *= alpha; }
        }

        // ---- O += P V: contraction over the tile's 32 keys, 128 output columns
#pragma unroll
        for (int kk = 0; kk < kQN / 16; ++kk) {
#pragma unroll
            for (int dp = 0; dp < kQD / 16; ++dp) {
                uint32_t b[4];
                ldsm_x4_t(vb + sw_off(kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dp * 2 + (lane >> 4)), b);
                mma_bf16(o[2 * dp], pa[kk], b[0], b[1]);
                mma_bf16(o[2 * dp + 1], pa[kk], b[2], b[3]);
            }
        }

        if (cc.last_of_item()) {
            // ---- O / l -> bf16 -> staging -> 16-byte stores; log-sum-exp
            // staging reuses this tile's K stage: every S = Q K^T of the block that reads it is
            // behind the barrier below, and the stage is refilled only after the next block barrier
            __syncthreads();
            unsigned char *stage = sK + st * kTileB + warp * (16 * kRowB);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                float l = l_run[hh];
                l += __shfl_xor_sync(0xffffffffu, l, 1);
                l += __shfl_xor_sync(0xffffffffu, l, 2);
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const int r = gid + 8 * hh;
#pragma unroll
                for (int i = 0; i < kQD / 8; ++i)
                    *reinterpret_cast<uint32_t *>(stage + sw_off(r, i) + tig * 4) = pack2(o[i][2 * hh] * inv, o[i][2 * hh + 1] * inv);
                const int rowq = warp * 16 + r;
                if (tig == 0 && rowq < cc.t.n_rows && p.lse)
                    p.lse[(int64_t)cc.h * p.total_tokens + cc.t.q_row + rowq] = l > 0.f ? (m_run[hh] + log2f(l)) * kLn2Q : -INFINITY;
            }
            __syncwarp();
            unsigned char *dst = p.out + ((int64_t)(cc.t.q_row + warp * 16) * p.n_heads + cc.h) * kRowB;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int idx = lane + 32 * i, r = idx >> 4, chunk = idx & 15;
                if (warp * 16 + r < cc.t.n_rows)
                    *reinterpret_cast<uint4 *>(dst + (int64_t)r * q_pitch + chunk * 16) =
                        *reinterpret_cast<const uint4 *>(stage + sw_off(r, chunk));
            }
            __syncwarp();
        }
        cc.next();
    }
    cp_async_wait<0>();
}

size_t prefill_qonly_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len)
{
    if (n_prompts < 0 || n_paths < 0 || max_pre_len < 0 || max_path_len < 0) return 256;
    return 256 + round_up((size_t)plan_max_tiles(0, n_paths, 0, max_path_len, kQM) * sizeof(TcTile), 256);
}

int launch_prefill_qonly(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                         const float *slopes, int n_heads, int n_kv_heads, float scale, void *out, float *lse,
                         void *ws, cudaStream_t st)
{
    TcHeader *hdr = static_cast<TcHeader *>(ws);
    TcTile *tiles = reinterpret_cast<TcTile *>(static_cast<char *>(ws) + 256);
    SP_CUDA(cudaMemsetAsync(ws, 0, 256, st));

    PlanArgs pa;
    pa.ppo = lay->prompt_path_off; pa.pre_start = lay->pre_start; pa.pre_len = lay->pre_len;
    pa.path_start = lay->path_start; pa.doc_len = lay->doc_len; pa.qry_len = lay->qry_len;
    pa.n_prompts = lay->n_prompts; pa.n_paths = lay->n_paths; pa.rows_mode = SP_ROWS_QUERY_ONLY; pa.tile_rows = kQM;
    pa.max_pre_len = lay->max_pre_len; pa.max_path_len = lay->max_path_len; pa.total_tokens = lay->total_tokens;
    pa.max_tiles = plan_max_tiles(lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len, kQM);
    pa.hdr = hdr; pa.tiles = tiles;
    prefill_plan_kernel<<<1, 1024, 0, st>>>(pa);
    SP_CUDA(cudaGetLastError());

    const int64_t items = plan_max_tiles(0, lay->n_paths, 0, lay->max_path_len, kQM) * n_heads;
    if (items == 0) return SP_OK;
    QoParams p;
    p.q = static_cast<const unsigned char *>(q); p.k = static_cast<const unsigned char *>(k);
    p.v = static_cast<const unsigned char *>(v); p.out = static_cast<unsigned char *>(out); p.lse = lse;
    p.hdr = hdr; p.tiles = tiles;
    p.n_heads = n_heads; p.n_kv_heads = n_kv_heads; p.kv_group = n_heads / n_kv_heads;
    p.total_tokens = lay->total_tokens; p.scale_log2e = scale * kLog2eQ;
    p.pos = pos; p.slopes = slopes;
    const int smem = (2 * kQStages + 1) * kTileB;
    const int grid = (int)std::min<int64_t>(items, (int64_t)kQBlocksPerSM * num_sms());
    if (pos) {
        SP_CUDA(cudaFuncSetAttribute(prefill_qonly_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_qonly_kernel<true><<<grid, kQThreads, smem, st>>>(p);
    } else {
        SP_CUDA(cudaFuncSetAttribute(prefill_qonly_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_qonly_kernel<false><<<grid, kQThreads, smem, st>>>(p);
    }
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

}  // namespace sp
