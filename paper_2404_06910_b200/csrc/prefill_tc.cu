// Fork-join prefill attention on the Blackwell tensor cores (bf16, head_dim 128).
// Section 3.2: a row attends to its prompt's preamble and, causally, to its own path.
//
// Work unit: (128-row query tile of one segment, head).  Its keys are the preamble's rows
// (all visible) followed by the segment's own rows up to the diagonal; key tiles that the
// fork-join mask excludes are never loaded or multiplied.  Per key tile of up to 64 keys:
//   S = Q K^T     tcgen05.mma, A and B from TMA-staged 128B-swizzled shared memory, fp32 in TMEM
//   P = softmax   4 warps, one thread per query row; two rolled passes over the tile in chunks of
//                 16 keys (tcgen05.ld): row maximum, then exp2 / sum with lazy rescaling, P rounded
//                 to bf16 and written over S in TMEM (tcgen05.st)
//   O += P V      tcgen05.mma with A = P from TMEM, B = V from shared memory (MN-major)
// Roles (warpgroups of 4 warps, registers rebalanced with setmaxnreg): warps 0-3 softmax,
// warps 4-7 epilogue (O / l -> bf16 -> global, LSE) off the softmax warps' critical path,
// warp 8 loads Q and K (TMA), warp 9 issues S = Q K^T and owns the TMEM allocation, warp 10 loads V
// (TMA) and cleans ragged V tiles, warp 11 issues O += P V.  The two products have an issuing thread
// each: one thread doing both was the busiest thread of the block (waits, work-list arithmetic and
// MMA issue back-pressure of two products in series), and every delay of it went straight into the
// softmax warps' wait for S.  The two threads' MMAs are ordered through mbarriers only where they
// touch the same tensor memory (S of tile g+2 overwrites P of tile g).
// K and V tiles are double-buffered in shared memory and S in TMEM, so the S = Q K^T of the next two
// tiles is issued while the softmax of the current tile runs.  The grid is persistent; two blocks
// share an SM (256 TMEM columns each).  A small plan kernel turns the ragged layout into a
// tile list.  Every mbarrier wait is bounded: on expiry the block records a timeout in the
// workspace status word, unwinds, frees its TMEM and exits.
// Compile-time variants: ALIBI adds the position bias to the scores; ROPE takes an unrotated Q and has the
// softmax warps rotate each query tile in shared memory before its first use (sp_superpose_prefill_rope).
#include <cstdlib>

#include "common.cuh"
#include "prefill_plan.cuh"
#include "tc_ptx.cuh"

namespace sp {

using namespace ptx;

constexpr int kBM = 128;              // query rows per tile
constexpr int kBN = 64;               // keys per tile
constexpr int kHD = 128;              // head_dim
constexpr int kTmaWarp = 8, kMmaWarp = 9, kCleanWarp = 10, kPvWarp = 11;
constexpr int kTcThreads = 12 * 32;   // warps 0-3 softmax, 4-7 epilogue, 8 Q/K loads, 9 S issuer, 10 V loads + cleaning, 11 P V issuer
constexpr int kQBytes = kBM * kHD * 2;     // 32 KB
constexpr int kKVBytes = kBN * kHD * 2;    // 16 KB per stage
constexpr int kTmemCols = 256;        // S/P double buffer: [0,64) [64,128)   O: [128,256)
constexpr int kCh = 16;               // keys per softmax chunk
constexpr float kLog2eT = 1.4426950408889634f;
constexpr float kLn2T = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;   // log2 units: rescale O only when the max grows by > 2^8

static_assert(kCh == 16, "the chunk loads and stores below are the 16-column forms");
__device__ __forceinline__ void tmem_ldc(uint32_t a, uint32_t (&r)[16]) { tmem_ld16(a, r); }
__device__ __forceinline__ void tmem_stc(uint32_t a, const uint32_t (&r)[8]) { tmem_st8(a, r); }

// The softmax warps run at the pace of their own instruction stream (one dependent chain per thread), so the
// three-input maximum and the two-lane fp32 forms below, which halve the instruction count of the row maximum,
// the scaling and the row sum, are worth a per cent of the kernel.
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// Packed pairs of fp32 (one 64-bit register): two lanes per FMA / ADD instruction.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Tiles with few valid rows are fetched through tensor maps with shorter boxes (32 or 64 rows
// instead of 128 / 64), so that ragged tails and query-only tiles do not pull in rows nobody
// needs.  A box lands as two swizzled halves of box_rows x 128 bytes each.
__device__ __host__ __forceinline__ int q_box_sel(int n_rows) { return n_rows <= 32 ? 0 : (n_rows <= 64 ? 1 : 2); }
__device__ __host__ __forceinline__ int kv_box_sel(int n_valid) { return n_valid <= 32 ? 0 : 1; }

struct TcParams {
    CUtensorMap mq[3], mk[2], mv[2];  // box rows: Q 32 / 64 / 128, K and V 32 / 64
    const TcHeader *hdr;
    const TcTile *tiles;
    uint32_t *status;
    __nv_bfloat16 *out;
    float *lse;
    int n_heads, kv_group;
    int64_t total_tokens;
    float scale_log2e;
    const float *pos, *slopes;        // ALiBi variant: token positions [T], head slopes [H]
    const float2 *rope_cs;            // ROPE variant: (cos, sin) of every (token, pair), [T][64]
    int rope_pairing;
    int stall_producer;               // test hook: the producer issues no load, so every wait runs out
};

// Key tile j of a query tile: preamble tiles first, then the segment's own rows up to the
// tile's last valid query row.
struct KvTile {
    int row0;        // packed row of the first key
    int n_valid;     // keys that exist (1..kBN)
    int k_off;       // own-segment offset of the first key; -1 for preamble tiles (no causal limit)
};
// Walks the block's work: items (query tile, head) in a grid-stride order, and inside an
// item its key tiles.  g counts key tiles since the block started: it selects the ring
// stage (g & 1) and the barrier parity ((g >> 1) & 1) of every double-buffered resource.
// Item number -> (query tile, head): heads vary fastest, so blocks running side by side read
// neighbouring 256-byte head slices of the same token rows.
__device__ __forceinline__ void item_decode(uint32_t it, uint32_t n_heads, uint32_t n_tiles, uint32_t &ti, int &h)
{
    (void)n_tiles;
    ti = it / n_heads;
    h = (int)(it - ti * n_heads);
}

struct Cursor {
    const TcTile *tiles;
    uint32_t it, n_items, n_tiles, stride, g, item_no;
    int n_heads, h, j, n_kv, n_pre;
    TcTile t;
    bool valid;
    __device__ __forceinline__ void load()
    {
        valid = it < n_items;
        if (valid) {
            uint32_t ti;
            item_decode(it, (uint32_t)n_heads, n_tiles, ti, h);
            t = tiles[ti];
            n_pre = (t.pre_len + kBN - 1) / kBN;
            n_kv = n_pre + (t.q_off + t.n_rows + kBN - 1) / kBN;
            j = 0;
        }
    }
    __device__ __forceinline__ KvTile kv() const
    {
        KvTile k;
        if (j < n_pre) {
            k.row0 = t.pre_row + j * kBN; k.n_valid = min(kBN, t.pre_len - j * kBN); k.k_off = -1;
        } else {
            const int o = (j - n_pre) * kBN;
            k.row0 = t.own_row + o; k.n_valid = min(kBN, t.q_off + t.n_rows - o); k.k_off = o;
        }
        return k;
    }
    __device__ __forceinline__ void init(const TcTile *tl, uint32_t n, int heads)
    {
        tiles = tl; n_items = n; n_heads = heads; n_tiles = n / (uint32_t)heads; it = blockIdx.x; stride = gridDim.x; g = 0; item_no = 0;
        load();
    }
    __device__ __forceinline__ void next()
    {
        ++g;
        if (++j == n_kv) { it += stride; ++item_no; load(); }
    }
    __device__ __forceinline__ bool last_of_item() const { return j == n_kv - 1; }
};

// S_FULL[st] (S = Q K^T of a tile complete) also tells the Q/K loader that K stage st is free;
// O_DONE[st] (O += P V complete) also frees V stage st for the V loader and the S / P columns st for
// the S issuer: one tcgen05.commit serves all waiters.
// L_READY[item parity]: the softmax warps have published an item's row sums; X_FREE[item parity]:
// the epilogue warps have read them, so the slot may be rewritten two items later.  Both are
// per-parity pairs because warps whose rows are masked out of a tile finish it almost at once:
// with a single barrier their arrivals for the next one-tile item could complete the phase of
// the current item before the warp on the diagonal has published its rows.
// O_FREE: the epilogue warps have read the item's O out of tensor memory, so the next item's
// first O = P V may overwrite it.
// V_CLEAN[st]: on a tile whose key count is not a multiple of 16, the rows of the V stage between the
// last key and the end of the last 16-key MMA step have been zeroed (see the cleaner role).
// Every thread that waits on a double-buffered barrier waits on each of its fills in order and is one of
// the parties the next fill depends on (the V loader is also the cleaner; the S issuer's wait for
// O_DONE gates the S whose softmax gates the next O += P V): a waiter that skipped fills could be two
// ahead, one that nothing waits for could fall two behind, and a parity wait would then answer for the
// wrong fill.
enum { BAR_Q_FULL = 0, BAR_Q_EMPTY, BAR_K_FULL, BAR_V_FULL = BAR_K_FULL + 2, BAR_S_FULL = BAR_V_FULL + 2,
       BAR_P_FULL = BAR_S_FULL + 2, BAR_O_DONE = BAR_P_FULL + 2, BAR_L_READY = BAR_O_DONE + 2,
       BAR_X_FREE = BAR_L_READY + 2, BAR_O_FREE = BAR_X_FREE + 2, BAR_V_CLEAN, BAR_Q_ROT = BAR_V_CLEAN + 2, BAR_DRAIN,
       BAR_COUNT = BAR_DRAIN + 2 };      // DRAIN: one per issuing thread

template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// ALIBI: scores get -slope_h * |pos_q - pos_k| before the softmax (Section 3.2.2: real-valued
// positions are no obstacle for ALiBi); the plain instantiation carries none of that code.
// ROPE: Q arrives unrotated; the softmax warps rotate each query tile in shared memory, at the tokens' real-valued
// positions (Section 3.2.2, footnote on RoPE), between its arrival and the item's first S = Q K^T.
template <bool ALIBI, bool ROPE>
__global__ void __launch_bounds__(kTcThreads, 2) prefill_tc_kernel(const __grid_constant__ TcParams p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char *sQ = smem;                                   // 128 rows x 128 cols, two 64-col halves
    unsigned char *sK = smem + kQBytes;                         // [2 stages] 64 keys x 128 cols
    unsigned char *sV = sK + 2 * kKVBytes;                      // [2 stages]
    unsigned char *sO = sV + 2 * kKVBytes;                      // [4 warps] 32 rows x 64 bytes, output staging
    __shared__ uint64_t bars[BAR_COUNT];
    __shared__ uint32_t tmem_base_s;
    __shared__ float x_l[2][kBM];                               // [item parity][row] row sums
    __shared__ float x_m[2][kBM];                               // [item parity][row] reference maxima

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < BAR_COUNT; ++i)
            mbar_init(&bars[i], ((i >= BAR_P_FULL && i < BAR_P_FULL + 2) || (i >= BAR_L_READY && i <= BAR_O_FREE) || i == BAR_Q_ROT) ? 128 : 1);
        fence_mbar_init();
        for (int i = 0; i < 3; ++i) prefetch_tmap(&p.mq[i]);
        for (int i = 0; i < 2; ++i) { prefetch_tmap(&p.mk[i]); prefetch_tmap(&p.mv[i]); }
    }
    if (warp == kMmaWarp) { tmem_alloc(&tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s;                            // S0 [0,64) S1 [64,128) O [128,256)
    const uint32_t n_items = p.hdr->n_tiles * (uint32_t)p.n_heads;
    bool ok = true;

    if (warp >= 8) {
        reg_dealloc<56>();              // warps 8-11: the two loaders and the two MMA issuers
        if (warp == kTmaWarp) {
            // -------------------------------------------------------------- Q and K loads (TMA)
            if (lane == 0) {
                uint32_t nq = 0, nk[2] = {0, 0};     // loads issued per "full" barrier
                // a query tile is read once: its lines may leave L2 first, which leaves more room for the K / V
                // rows that the other query tiles of the path read again
                const uint64_t pol_first = l2_policy_evict_first();
                Cursor c;
#pragma unroll 1
                for (c.init(p.tiles, n_items, p.n_heads); c.valid && ok && !p.stall_producer; c.next()) {
                    const int hk = c.h / p.kv_group;
                    const KvTile kt = c.kv();
                    const int st = c.g & 1;
                    const uint32_t ph = (c.g >> 1) & 1;
                    if (!(ok = mbar_wait(&bars[BAR_S_FULL + st], ph ^ 1))) break;       // K stage free
                    const int ks = kv_box_sel(kt.n_valid);
                    mbar_expect_tx(&bars[BAR_K_FULL + st], (32u << ks) * (kHD * 2));
                    tma_load_3d(sK + st * kKVBytes, &p.mk[ks], 0, kt.row0, hk * 2, &bars[BAR_K_FULL + st]);
                    ++nk[st];
                    if (c.j == 0) {
                        // the item's query tile, after its first K tile: the Q slot is the later of the two to come free
                        if (!(ok = mbar_wait(&bars[BAR_Q_EMPTY], (c.item_no & 1) ^ 1))) break;
                        const int qs = q_box_sel(c.t.n_rows);
                        mbar_expect_tx(&bars[BAR_Q_FULL], (32u << qs) * (kHD * 2));
                        tma_load_3d_hint(sQ, &p.mq[qs], 0, c.t.q_row, c.h * 2, &bars[BAR_Q_FULL], pol_first);
                        ++nq;
                    }
                }
                if (!ok) {
                    // a wait ran out: before the block may exit, its own copies in flight must
                    // have landed (bounded waits on the phase of the last load of each buffer)
                    if (nq) mbar_wait(&bars[BAR_Q_FULL], (nq - 1) & 1);
                    for (int st = 0; st < 2; ++st)
                        if (nk[st]) mbar_wait(&bars[BAR_K_FULL + st], (nk[st] - 1) & 1);
                }
            }
        } else if (warp == kMmaWarp) {
            // -------------------------------------------------------------- MMA issuer, S = Q K^T
            if (lane == 0) {
                // Descriptor words are loop-invariant up to a small address offset: build them once.
                // High word: stride-dimension offset 1024 B (8-row groups), descriptor version 1, 128B swizzle.
                const uint32_t d_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
                const uint32_t q_lo = ((smem_u32(sQ) & 0x3ffffu) >> 4) | (1u << 16);
                const uint32_t k_lo = ((smem_u32(sK) & 0x3ffffu) >> 4) | (1u << 16);
                Cursor cs;                          // next S = Q K^T to issue
#pragma unroll 1
                for (cs.init(p.tiles, n_items, p.n_heads); cs.valid && ok; cs.next()) {
                    const uint32_t st = cs.g & 1;
                    if (cs.j == 0 && !(ok = mbar_wait(&bars[ROPE ? BAR_Q_ROT : BAR_Q_FULL], cs.item_no & 1))) break;
                    if (!(ok = mbar_wait(&bars[BAR_K_FULL + st], (cs.g >> 1) & 1))) break;
                    // S(g) lands on the columns of P(g-2): the O += P V that reads them (issued by the other
                    // issuing thread) must be complete
                    if (cs.g >= 2 && !(ok = mbar_wait(&bars[BAR_O_DONE + st], ((cs.g >> 1) - 1) & 1))) break;
                    tc_fence_after();
                    const int n_valid = cs.kv().n_valid;
                    const int n_mma = (n_valid + 15) & ~15;
                    const uint32_t id_s = idesc_bf16(kBM, 0, 0, 0) | ((uint32_t)(n_mma >> 3) << 17);
                    const uint32_t kb = k_lo + st * (kKVBytes >> 4);
                    const uint32_t d = tb + st * kBN;
                    // second 64-column half of a box: box_rows x 128 bytes further on (in 16-byte units)
                    const uint32_t q_half = (32u << q_box_sel(cs.t.n_rows)) * 8u;
                    const uint32_t k_half = (32u << kv_box_sel(n_valid)) * 8u;
#pragma unroll
                    for (int kk = 0; kk < kHD / 16; ++kk)              // contraction over head_dim
                        umma_ss_lh(d, q_lo + (kk >> 2) * q_half + (kk & 3) * 2,
                                   kb + (kk >> 2) * k_half + (kk & 3) * 2, d_hi, id_s, kk > 0 ? 1u : 0u);
                    umma_commit(&bars[BAR_S_FULL + st]);
                    if (cs.last_of_item()) umma_commit(&bars[BAR_Q_EMPTY]);
                }
                if (!ok) {
                    // a wait ran out: let every MMA this thread issued finish (bounded) before the
                    // tensor memory they write is freed
                    umma_commit(&bars[BAR_DRAIN]);
                    mbar_wait(&bars[BAR_DRAIN], 0);
                }
            }
        } else if (warp == kPvWarp) {
            // -------------------------------------------------------------- MMA issuer, O += P V
            if (lane == 0) {
                const uint32_t d_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
                const uint32_t v_lo = (smem_u32(sV) & 0x3ffffu) >> 4;     // leading-dimension offset (half stride) added per tile
                const uint32_t id_o = idesc_bf16(kBM, kHD, 0, 1);
                uint32_t n_ragged[2] = {0, 0};      // ragged tiles seen per V stage (phase of V_CLEAN)
                Cursor cp;
#pragma unroll 1
                for (cp.init(p.tiles, n_items, p.n_heads); cp.valid && ok; cp.next()) {
                    const uint32_t st = cp.g & 1;
                    const uint32_t ph = (cp.g >> 1) & 1;
                    const int pv_valid = cp.kv().n_valid;
                    const int n_k = (pv_valid + 15) >> 4;                 // 16-key steps
                    // everything but P first: P is what arrives last
                    if (!(ok = mbar_wait(&bars[BAR_V_FULL + st], ph))) break;
                    if ((pv_valid & 15) && !(ok = mbar_wait(&bars[BAR_V_CLEAN + st], n_ragged[st]++ & 1))) break;
                    // the first O = P V of an item overwrites O: the previous item's must have been read out
                    if (cp.j == 0 && cp.item_no > 0 && !(ok = mbar_wait(&bars[BAR_O_FREE], (cp.item_no - 1) & 1))) break;
                    const uint32_t vb = (v_lo + st * (kKVBytes >> 4)) | (((32u << kv_box_sel(pv_valid)) * 8u) << 16);
                    const uint32_t pa = tb + st * kBN;
                    if (!(ok = mbar_wait(&bars[BAR_P_FULL + st], ph))) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < kBN / 16; ++kk)                 // contraction over keys
                        if (kk < n_k)
                            umma_ts_lh(tb + 128, pa + kk * 8, vb + kk * (2048 >> 4), d_hi, id_o, (cp.j > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(&bars[BAR_O_DONE + st]);
                }
                if (!ok) {
                    umma_commit(&bars[BAR_DRAIN + 1]);
                    mbar_wait(&bars[BAR_DRAIN + 1], 0);
                }
            }
        } else if (warp == kCleanWarp) {
            // -------------------------------------------------------------- V loader and cleaner
            auto clean_tile = [&](uint32_t g, int n_valid) -> bool {
                const int st = g & 1;
                if (!mbar_wait_warp(&bars[BAR_V_FULL + st], (g >> 1) & 1)) return false;
                if ((n_valid & 15) == 0) return true;
                const int n_mma = (n_valid + 15) & ~15;
                const int half_bytes = (32 << kv_box_sel(n_valid)) * 128;      // one 64-column half of the box
                unsigned char *vs = sV + st * kKVBytes;
                // (rows n_valid .. n_mma-1) x 2 halves x 8 pieces of 16 bytes; the 128-byte swizzle only
                // permutes the pieces inside a row
                for (int i = lane; i < (n_mma - n_valid) * 16; i += 32) {
                    const int r = n_valid + (i >> 4), half = (i >> 3) & 1, piece = i & 7;
                    *reinterpret_cast<uint4 *>(vs + half * half_bytes + r * 128 + piece * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async();                 // generic-proxy stores -> visible to the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[BAR_V_CLEAN + st]);
                return true;
            };
            // O += P V contracts over the keys rounded up to 16.  The rows of the V stage past the
            // tile's last key hold whatever follows in the packed tensor (another path's rows);
            // their P is exactly zero, but 0 x Inf or 0 x NaN would still reach O.  This warp
            // zeroes those rows before the issuer may use the stage, so a path's output depends on
            // nothing outside its own keys (Section 3.2: paths do not see each other).
            // The same warp loads V: tile t goes into its stage as soon as O += P V of tile t-2 (the
            // stage's previous user) is complete, then tile t-1, loaded one turn earlier, is waited for and
            // cleaned.  Loading and cleaning in one thread keeps every V barrier's waits in fill order.
            Cursor c;
            int prev_valid = 0;                   // keys of tile t-1; 0: no such tile
            uint32_t t_issued = 0;
            c.init(p.tiles, n_items, p.n_heads);
#pragma unroll 1
            while (ok && (c.valid || prev_valid)) {
                if (c.valid) {
                    const int st = c.g & 1;
                    if (c.g >= 2 && !(ok = mbar_wait_warp(&bars[BAR_O_DONE + st], ((c.g >> 1) - 1) & 1))) break;
                    const KvTile kt = c.kv();
                    if (lane == 0) {
                        const int ks = kv_box_sel(kt.n_valid);
                        mbar_expect_tx(&bars[BAR_V_FULL + st], (32u << ks) * (kHD * 2));
                        tma_load_3d(sV + st * kKVBytes, &p.mv[ks], 0, kt.row0, (c.h / p.kv_group) * 2, &bars[BAR_V_FULL + st]);
                    }
                    ++t_issued;
                    const int nv = kt.n_valid;
                    // tile t-1
                    if (prev_valid) ok = clean_tile(c.g - 1, prev_valid);
                    prev_valid = nv;
                    c.next();
                } else {
                    ok = clean_tile(c.g - 1, prev_valid);
                    prev_valid = 0;
                }
            }
            if (!ok && t_issued) {
                // a wait ran out: the V copies in flight must land before the block exits (bounded)
                mbar_wait_warp(&bars[BAR_V_FULL + ((t_issued - 1) & 1)], ((t_issued - 1) >> 1) & 1);
                if (t_issued >= 2) mbar_wait_warp(&bars[BAR_V_FULL + ((t_issued - 2) & 1)], ((t_issued - 2) >> 1) & 1);
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        // ------------------------------------------------------------------ softmax
        // One thread per query row.
        reg_alloc<104>();
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const float sc = p.scale_log2e;
        Cursor c;
        c.init(p.tiles, n_items, p.n_heads);
        float m_ref = -INFINITY, l = 0.f;          // reference maximum (log2 units) and row sum
        float pq = 0.f, slope_l2 = 0.f;            // ALiBi: this row's position, the head's slope (log2 units)
        const float sc_exp = ALIBI ? 1.f : sc;     // ALiBi scores are scaled when the bias is added

        while (c.valid && ok) {
            const int st = c.g & 1;
            const bool first = c.j == 0;
            const TcTile &t = c.t;
            const KvTile kt = c.kv();
            const uint32_t s_addr = tb + lane_addr + st * kBN;
            const int n_mma = (kt.n_valid + 15) & ~15;
            // keys this row / the warp's first and last rows may see
            const int lim = kt.k_off < 0 ? kt.n_valid : min(kt.n_valid, t.q_off + row - kt.k_off + 1);
            const int lim0 = kt.k_off < 0 ? kt.n_valid : min(kt.n_valid, t.q_off + warp * 32 - kt.k_off + 1);
            const int lim31 = kt.k_off < 0 ? kt.n_valid : min(kt.n_valid, t.q_off + warp * 32 + 31 - kt.k_off + 1);
            // A warp whose 32 rows lie past the tile's last valid row does no arithmetic at all:
            // its rows of P and O are never stored (it still takes part in every barrier).
            const bool live_w = warp * 32 < t.n_rows;
            if (first) {
                m_ref = -INFINITY; l = 0.f;
                if (ALIBI) {
                    pq = row < t.n_rows ? p.pos[t.q_row + row] : 0.f;
                    slope_l2 = p.slopes[c.h] * kLog2eT;
                }
            }
            // ALiBi: lane i fetches the positions of keys i and 32 + i of the tile (ahead of the wait,
            // off the chain); the chunk loops read them with shuffles instead of 64 loads per thread
            float kp0 = 0.f, kp1 = 0.f;
            if (ALIBI) {
                if (lane < kt.n_valid) kp0 = __ldg(p.pos + kt.row0 + lane);
                if (32 + lane < kt.n_valid) kp1 = __ldg(p.pos + kt.row0 + 32 + lane);
            }
            if (ROPE && first) {
                // This thread's row of the new query tile: 8 pieces of 16 bytes in each 64-column half (the 128-byte
                // swizzle permutes the pieces of a row by its index mod 8); the (cos, sin) pairs come from the
                // per-token table.  The arithmetic is the standalone rotation's, so the tile equals what that
                // kernel would have stored.
                if (!(ok = mbar_wait_warp(&bars[BAR_Q_FULL], c.item_no & 1))) break;
                if (row < t.n_rows) {
                    unsigned char *h0 = sQ + row * 128, *h1 = h0 + (32 << q_box_sel(t.n_rows)) * 128;
                    const float4 *tab = reinterpret_cast<const float4 *>(p.rope_cs + (int64_t)(t.q_row + row) * (kHD / 2));
                    const bool half_split = p.rope_pairing == SP_ROPE_HALF_SPLIT;
#pragma unroll 1
                    for (int pc = 0; pc < 8; ++pc) {
                        uint4 *pa = reinterpret_cast<uint4 *>(h0 + ((pc ^ (row & 7)) << 4));
                        uint4 *pb = reinterpret_cast<uint4 *>(h1 + ((pc ^ (row & 7)) << 4));
                        uint4 va = *pa, vb = *pb;
                        uint32_t *ua = reinterpret_cast<uint32_t *>(&va), *ub = reinterpret_cast<uint32_t *>(&vb);
                        if (half_split) {            // element j of the piece in half 0 pairs with element j in half 1
#pragma unroll
                            for (int j2 = 0; j2 < 4; ++j2) {
                                const float4 w = __ldg(tab + pc * 4 + j2);      // pairs 8 pc + 2 j2, + 1
                                const float a0 = __uint_as_float(ua[j2] << 16), a1 = __uint_as_float(ua[j2] & 0xffff0000u);
                                const float b0 = __uint_as_float(ub[j2] << 16), b1 = __uint_as_float(ub[j2] & 0xffff0000u);
                                float na0, nb0, na1, nb1;
                                rope_rotate(a0, b0, w.x, w.y, na0, nb0);
                                rope_rotate(a1, b1, w.z, w.w, na1, nb1);
                                ua[j2] = pack_bf16x2(na0, na1);
                                ub[j2] = pack_bf16x2(nb0, nb1);
                            }
                        } else {                     // neighbours pair up: pair 4 pc + j2 in half 0, 32 + 4 pc + j2 in half 1
#pragma unroll
                            for (int j2 = 0; j2 < 4; j2 += 2) {
                                const float4 wa = __ldg(tab + pc * 2 + (j2 >> 1)), wb = __ldg(tab + 16 + pc * 2 + (j2 >> 1));
                                float n0, n1;
                                rope_rotate(__uint_as_float(ua[j2] << 16), __uint_as_float(ua[j2] & 0xffff0000u), wa.x, wa.y, n0, n1);
                                ua[j2] = pack_bf16x2(n0, n1);
                                rope_rotate(__uint_as_float(ua[j2 + 1] << 16), __uint_as_float(ua[j2 + 1] & 0xffff0000u), wa.z, wa.w, n0, n1);
                                ua[j2 + 1] = pack_bf16x2(n0, n1);
                                rope_rotate(__uint_as_float(ub[j2] << 16), __uint_as_float(ub[j2] & 0xffff0000u), wb.x, wb.y, n0, n1);
                                ub[j2] = pack_bf16x2(n0, n1);
                                rope_rotate(__uint_as_float(ub[j2 + 1] << 16), __uint_as_float(ub[j2 + 1] & 0xffff0000u), wb.z, wb.w, n0, n1);
                                ub[j2 + 1] = pack_bf16x2(n0, n1);
                            }
                        }
                        *pa = va; *pb = vb;
                    }
                }
                fence_proxy_async();                 // generic-proxy stores -> visible to the MMA's reads
                mbar_arrive(&bars[BAR_Q_ROT]);
            }
            if (!(ok = mbar_wait_warp(&bars[BAR_S_FULL + st], (c.g >> 1) & 1))) break;
            tc_fence_after();

            // The tile is walked twice in chunks of 16 keys (rolled loops, scores re-read from tensor
            // memory): the code of this role stays small, which matters more than the second read.
            // n_ch chunks are read by the MMA; `see` of them hold keys some row of this warp may see.
            const int n_ch = (n_mma + kCh - 1) / kCh;
            const int see = live_w ? min(n_ch, (max(lim31, 0) + kCh - 1) / kCh) : 0;
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
            for (int ch = 0; ch < see; ++ch) {          // pass 1: the row's maximum over the tile
                uint32_t r[kCh];
                tmem_ldc(s_addr + ch * kCh, r);
                tmem_ld_wait();
                if (ALIBI) {            // score * scale - slope * |distance|; key positions come from the lanes' registers
                    const float kp = ch < 2 ? kp0 : kp1;
#pragma unroll
                    for (int i = 0; i < kCh; ++i) {
                        const float pk = __shfl_sync(0xffffffffu, kp, (ch & 1) * kCh + i);
                        r[i] = __float_as_uint(fmaf(__uint_as_float(r[i]), sc, -slope_l2 * fabsf(pq - pk)));
                    }
                    tmem_st16(s_addr + ch * kCh, r);     // the biased scores replace the raw ones: pass 2 reads them as they are
                }
                // keys past the row's limit (causal diagonal, ragged tail) -> -inf; skipped when the
                // whole warp sees the whole chunk
                if (ch * kCh + 16 > lim0) {
#pragma unroll
                    for (int i = 0; i < kCh; ++i) r[i] = (ch * kCh + i < lim) ? r[i] : 0xff800000u;
                }
#pragma unroll
                for (int i = 0; i < kCh; i += 2) mx[(i >> 1) & 3] = fmax3(mx[(i >> 1) & 3], __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
            }
            if (ALIBI) tmem_st_wait();                  // the biased scores are in place before pass 2 reads them
            const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * sc_exp;
            float alpha = 1.f;
            bool grow = false;
            if (first) {
                m_ref = m_tile;
            } else if (m_tile > m_ref + kRescaleThreshold) {
                alpha = ex2(m_ref - m_tile);
                m_ref = m_tile;
                grow = true;
            }
            if (__any_sync(0xffffffffu, grow)) {     // rare: bring O and l to the new reference
                // needs the previous tile's O += P V complete
                if (!(ok = mbar_wait_warp(&bars[BAR_O_DONE + ((c.g - 1) & 1)], ((c.g - 1) >> 1) & 1))) break;
                tc_fence_after();
                l *= alpha;
#pragma unroll 1
                for (int cc = 0; cc < kHD / 32; ++cc) {
                    uint32_t o[32];
                    tmem_ld32(tb + lane_addr + 128 + cc * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st32(tb + lane_addr + 128 + cc * 32, o);
                }
            }
            if (live_w) {
                // masked scores are -inf, so exp2 gives exactly 0 for them
                const float nm = -m_ref;
                uint64_t rs2[4] = {0ull, 0ull, 0ull, 0ull};      // packed pairs of partial row sums
                const uint64_t sc2 = pack_f32x2(sc_exp, sc_exp), nm2 = pack_f32x2(nm, nm);
#pragma unroll 1
                for (int ch = 0; ch < n_ch; ++ch) {     // pass 2: P = exp2(score - reference) as bf16, written over S
                    uint32_t pk[kCh / 2];
                    if (ch < see) {
                        uint32_t r[kCh];
                        tmem_ldc(s_addr + ch * kCh, r);
                        tmem_ld_wait();
                        if (ch * kCh + 16 > lim0) {
#pragma unroll
                            for (int i = 0; i < kCh; ++i) r[i] = (ch * kCh + i < lim) ? r[i] : 0xff800000u;
                        }
#pragma unroll
                        for (int i = 0; i < kCh; i += 2) {
                            float x0, x1;
                            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2), x0, x1);
                            const float p0 = ex2(x0), p1 = ex2(x1);
                            rs2[(i >> 1) & 3] = add_f32x2(rs2[(i >> 1) & 3], pack_f32x2(p0, p1));
                            pk[i >> 1] = pack_bf16x2(p0, p1);
                        }
                    } else {                            // keys no row of this warp sees
#pragma unroll
                        for (int i = 0; i < kCh / 2; ++i) pk[i] = 0u;
                    }
                    // P chunk ch (8 columns of bf16 pairs) lands on score columns already consumed
                    tmem_stc(s_addr + ch * (kCh / 2), pk);
                }
                {
                    float a0, a1;
                    unpack_f32x2(add_f32x2(add_f32x2(rs2[0], rs2[1]), add_f32x2(rs2[2], rs2[3])), a0, a1);
                    l += a0 + a1;
                }
            }
            // P of this tile is in TMEM: release the tile to the MMA issuer
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&bars[BAR_P_FULL + st]);
            if (c.last_of_item()) {                 // hand the item's row statistics to the epilogue warps
                const uint32_t xp = c.item_no & 1;
                // the slot was last used two items ago: the epilogue must have read it
                if (c.item_no >= 2 && !(ok = mbar_wait_warp(&bars[BAR_X_FREE + xp], ((c.item_no >> 1) - 1) & 1))) break;
                x_l[xp][row] = l;
                x_m[xp][row] = m_ref;
                mbar_arrive(&bars[BAR_L_READY + xp]);
            }
            c.next();
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 4-7)
        // O / l -> bf16 -> global and the log-sum-exp, off the softmax warps' critical path.
        const int quad = warp - 4;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        unsigned char *stage = sO + quad * 2048;
        const int64_t row_pitch = (int64_t)p.n_heads * kHD * 2;
        uint32_t g_end = 0, item_no = 0;
        for (uint32_t it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++item_no) {
            uint32_t ti;
            int h;
            item_decode(it, (uint32_t)p.n_heads, p.hdr->n_tiles, ti, h);
            const TcTile t = p.tiles[ti];
            g_end += (t.pre_len + kBN - 1) / kBN + (t.q_off + t.n_rows + kBN - 1) / kBN;
            const uint32_t g_last = g_end - 1;
            const int xp = item_no & 1;
            if (!(ok = mbar_wait_warp(&bars[BAR_L_READY + xp], (item_no >> 1) & 1))) break;
            const float l_row = x_l[xp][row], m_row = x_m[xp][row];
            mbar_arrive(&bars[BAR_X_FREE + xp]);
            if (!(ok = mbar_wait_warp(&bars[BAR_O_DONE + (g_last & 1)], (g_last >> 1) & 1))) break;   // last O += P V
            tc_fence_after();
            const float inv = 1.f / l_row;
            unsigned char *dst = reinterpret_cast<unsigned char *>(p.out) + ((int64_t)t.q_row * p.n_heads + h) * (kHD * 2);
            const bool live_w = quad * 32 < t.n_rows;
#pragma unroll 1
            for (int cc = 0; cc < kHD / 32; ++cc) {
                uint32_t ro[32];
                if (live_w) {
                    tmem_ld32(tb + lane_addr + 128 + cc * 32, ro);
                    tmem_ld_wait();
                }
                if (cc == kHD / 32 - 1) {              // O is in registers: the accumulator may be overwritten
                    tc_fence_before();
                    mbar_arrive(&bars[BAR_O_FREE]);
                }
                if (live_w) {
                    // thread = row -> shared staging (xor-swizzled 16-byte pieces) -> each store
                    // instruction writes 8 rows x 64 contiguous bytes
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(ro[q4 * 8 + 0]) * inv, __uint_as_float(ro[q4 * 8 + 1]) * inv);
                        w.y = pack_bf16x2(__uint_as_float(ro[q4 * 8 + 2]) * inv, __uint_as_float(ro[q4 * 8 + 3]) * inv);
                        w.z = pack_bf16x2(__uint_as_float(ro[q4 * 8 + 4]) * inv, __uint_as_float(ro[q4 * 8 + 5]) * inv);
                        w.w = pack_bf16x2(__uint_as_float(ro[q4 * 8 + 6]) * inv, __uint_as_float(ro[q4 * 8 + 7]) * inv);
                        *reinterpret_cast<uint4 *>(stage + lane * 64 + ((q4 ^ ((lane >> 1) & 3)) << 4)) = w;
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rr = (lane >> 2) + 8 * i, piece = lane & 3;
                        const uint4 w = *reinterpret_cast<const uint4 *>(stage + rr * 64 + ((piece ^ ((rr >> 1) & 3)) << 4));
                        if (quad * 32 + rr < t.n_rows)            // streaming store: the output is not read again here
                            __stcs(reinterpret_cast<uint4 *>(dst + (int64_t)(quad * 32 + rr) * row_pitch + cc * 64 + piece * 16), w);
                    }
                    __syncwarp();
                }
            }
            if (row < t.n_rows && p.lse)
                p.lse[(int64_t)h * p.total_tokens + t.q_row + row] = (m_row + log2f(l_row)) * kLn2T;
        }
    }

    if (!ok && lane == 0) atomicExch(p.status, (uint32_t)STATUS_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tb, kTmemCols);
}

// ---- host side ---------------------------------------------------------------------------
// Failure-detection test hook (host-injected, no GPU fault): while set, the producer loads no
// tile, every bounded wait expires, the blocks unwind and the call reports SP_ERR_TIMEOUT
// through the workspace status word.  Set only through sp_test_stall_producer(), a symbol for
// the test suite that the public header does not declare.
static bool g_stall_producer = false;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int encode_rows_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int box_rows)
{
    // [rows, cols] bf16 row-major seen as 3-D (64 columns, rows, cols / 64): one box = box_rows x
    // 128 columns of one head, delivered as two 128-byte-swizzled halves [half][row][64 columns],
    // which is the layout the MMA descriptors expect -- one TMA instruction per tile.
    cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, 128};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    SP_REQUIRE(r == CUDA_SUCCESS, SP_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return SP_OK;
}

// The same view for the other TMA-fed kernels of the library.
int make_rows_tensor_map(CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int box_rows)
{
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SP_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        SP_REQUIRE(fn != nullptr && qres == cudaDriverEntryPointSuccess, SP_ERR_CUDA,
                   "cuTensorMapEncodeTiled is not available from this driver");
        enc = reinterpret_cast<EncodeTiledFn>(fn);
    }
    return encode_rows_map(enc, m, base, rows, cols, box_rows);
}
bool prefill_stall_hook() { return g_stall_producer; }
int launch_prefill_pair(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                        const float *slopes, int n_heads, int n_kv_heads, float scale, void *out, float *lse,
                        void *ws, cudaStream_t st);

static int64_t max_tiles(int n_prompts, int n_paths, int max_pre_len, int max_path_len)
{
    return plan_max_tiles(n_prompts, n_paths, max_pre_len, max_path_len, kBM);
}

size_t prefill_tc_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len, int)
{
    if (n_prompts < 0 || n_paths < 0 || max_pre_len < 0 || max_path_len < 0) return 256;
    const size_t cap = (size_t)max_tiles(n_prompts, n_paths, max_pre_len, max_path_len);
    return 256 + round_up(cap * sizeof(TcTile), 256) + round_up(cap * sizeof(PairRec), 256);
}

static int launch_tc(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                     const float *slopes, const float2 *rope_cs, int rope_pairing, int n_heads, int n_kv_heads,
                     float scale, int rows, void *out, float *lse, void *ws, cudaStream_t st);

int launch_prefill_tc(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                      const float *slopes, int n_heads, int n_kv_heads, float scale, int rows, void *out,
                      float *lse, void *ws, size_t, cudaStream_t st)
{
    return launch_tc(q, k, v, lay, pos, slopes, nullptr, 0, n_heads, n_kv_heads, scale, rows, out, lse, ws, st);
}

// The (cos, sin) table of the ROPE variant sits behind the tile list and the pair list.
size_t prefill_tc_rope_workspace_bytes(int n_prompts, int n_paths, int max_pre_len, int max_path_len, int64_t total_tokens)
{
    return prefill_tc_workspace_bytes(n_prompts, n_paths, max_pre_len, max_path_len, 0) +
           round_up((size_t)std::max<int64_t>(total_tokens, 0) * (kHD / 2) * sizeof(float2), 256);
}

int launch_prefill_tc_rope(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos, double base,
                           int pairing, int n_heads, int n_kv_heads, float scale, void *out, float *lse, void *ws,
                           cudaStream_t st)
{
    float2 *table = reinterpret_cast<float2 *>(static_cast<char *>(ws) + prefill_tc_workspace_bytes(
                        lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len, 0));
    if (int rc = launch_rope_table(pos, lay->total_tokens, kHD, base, table, st)) return rc;
    return launch_tc(q, k, v, lay, nullptr, nullptr, table, pairing, n_heads, n_kv_heads, scale, SP_ROWS_ALL, out, lse, ws, st);
}

static int launch_tc(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                     const float *slopes, const float2 *rope_cs, int rope_pairing, int n_heads, int n_kv_heads,
                     float scale, int rows, void *out, float *lse, void *ws, cudaStream_t st)
{
    {
        // Experimental variant (two query tiles of a segment per block, shared K/V stages; prefill_pair.cu).
        // Parity-green and slower than this kernel on every workload measured, so it is off unless
        // SP_B200_PREFILL_PAIR=1 is set when the library is first used.
        static const bool use_pair = [] { const char *e = std::getenv("SP_B200_PREFILL_PAIR"); return e && e[0] == '1'; }();
        if (use_pair && rows == SP_ROWS_ALL && !rope_cs)
            return launch_prefill_pair(q, k, v, lay, pos, slopes, n_heads, n_kv_heads, scale, out, lse, ws, st);
    }
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SP_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        SP_REQUIRE(fn != nullptr && qres == cudaDriverEntryPointSuccess, SP_ERR_CUDA,
                   "cuTensorMapEncodeTiled is not available from this driver");
        enc = reinterpret_cast<EncodeTiledFn>(fn);
    }
    SP_REQUIRE(((int64_t)n_heads * kHD * 2) % 16 == 0, SP_ERR_INVALID_ARG, "row stride must be a multiple of 16 bytes");

    TcParams p;
    for (int i = 0; i < 3; ++i)
        if (int rc = encode_rows_map(enc, &p.mq[i], q, lay->total_tokens, (int64_t)n_heads * kHD, 32 << i)) return rc;
    for (int i = 0; i < 2; ++i) {
        if (int rc = encode_rows_map(enc, &p.mk[i], k, lay->total_tokens, (int64_t)n_kv_heads * kHD, 32 << i)) return rc;
        if (int rc = encode_rows_map(enc, &p.mv[i], v, lay->total_tokens, (int64_t)n_kv_heads * kHD, 32 << i)) return rc;
    }

    TcHeader *hdr = static_cast<TcHeader *>(ws);
    TcTile *tiles = reinterpret_cast<TcTile *>(static_cast<char *>(ws) + 256);
    SP_CUDA(cudaMemsetAsync(ws, 0, 256, st));

    PlanArgs pa;
    pa.ppo = lay->prompt_path_off; pa.pre_start = lay->pre_start; pa.pre_len = lay->pre_len;
    pa.path_start = lay->path_start; pa.doc_len = lay->doc_len; pa.qry_len = lay->qry_len;
    pa.n_prompts = lay->n_prompts; pa.n_paths = lay->n_paths; pa.rows_mode = rows; pa.tile_rows = kBM;
    pa.max_pre_len = lay->max_pre_len; pa.max_path_len = lay->max_path_len; pa.total_tokens = lay->total_tokens;
    pa.max_tiles = plan_max_tiles(lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len, kBM);
    pa.hdr = hdr; pa.tiles = tiles;
    prefill_plan_kernel<<<1, 1024, 0, st>>>(pa);
    SP_CUDA(cudaGetLastError());

    p.hdr = hdr; p.tiles = tiles; p.status = &hdr->status;
    p.out = static_cast<__nv_bfloat16 *>(out); p.lse = lse;
    p.n_heads = n_heads; p.kv_group = n_heads / n_kv_heads;
    p.total_tokens = lay->total_tokens; p.scale_log2e = scale * kLog2eT;
    p.pos = pos; p.slopes = slopes;
    p.rope_cs = rope_cs; p.rope_pairing = rope_pairing;
    p.stall_producer = g_stall_producer ? 1 : 0;      // test hook, see sp_test_stall_producer below

    const int64_t items = max_tiles(lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len) * n_heads;
    if (items == 0) return SP_OK;
    const int grid = (int)std::min<int64_t>(items, 2 * num_sms());
    const int smem = kQBytes + 4 * kKVBytes + 4 * 2048 + 1024;
    if (rope_cs) {
        SP_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_tc_kernel<false, true><<<grid, kTcThreads, smem, st>>>(p);
    } else if (pos) {
        SP_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_tc_kernel<true, false><<<grid, kTcThreads, smem, st>>>(p);
    } else {
        SP_CUDA(cudaFuncSetAttribute(prefill_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_tc_kernel<false, false><<<grid, kTcThreads, smem, st>>>(p);
    }
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

}  // namespace sp

extern "C" void sp_test_stall_producer(int on) { sp::g_stall_producer = on != 0; }
