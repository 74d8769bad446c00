// Fork-join prefill attention on the Blackwell tensor cores, two query tiles per block
// (bf16, head_dim 128).  Section 3.2: a row attends to its prompt's preamble and, causally, to its
// own path.
//
// One block per SM works on a PAIR of consecutive 128-row query tiles of one segment and one head
// (a segment's last tile may have no partner).  The two tiles read the same key tiles -- the
// preamble's and the segment's own rows up to the first tile's diagonal -- so those K and V tiles
// are fetched into shared memory once and used by both.  Each tile of the pair is a "lane" with the
// roles of the single-tile kernel (prefill_tc.cu): its own Q buffer, S/P double buffer and O
// accumulator in tensor memory, softmax warpgroup, epilogue warpgroup and MMA-issuing thread.
// Shared by both lanes: the TMA producer, a ring of kNS K and V stages, the V cleaner.
// A stage is used by lane 0, lane 1 or both; it is handed back to the producer when both lanes
// have released it: the lane that multiplies with it releases it by tcgen05.commit, the other lane
// by a plain arrival of its issuing thread when it passes the stage.  Every thread that waits on a
// ring barrier waits on every fill in order and is one of the parties the stage's release needs, so
// none can be a fill ahead of, or behind, the barrier it asks (a parity wait cannot tell fills two
// apart).
#include "common.cuh"
#include "prefill_plan.cuh"
#include "tc_ptx.cuh"

namespace sp {

using namespace ptx;

namespace pair {

constexpr int kBM = 128;              // query rows per tile
constexpr int kBN = 64;               // keys per tile
constexpr int kHD = 128;              // head_dim
constexpr int kNS = 4;                // K / V ring stages
constexpr int kLaneWarps = 12;        // per lane: 0-3 softmax, 4-7 epilogue, 8 producer (lane 0), 9 MMA issuer, 10 V cleaner (lane 0), 11 idle
constexpr int kThreads = 2 * kLaneWarps * 32;
constexpr int kQBytes = kBM * kHD * 2;     // 32 KB
constexpr int kKVBytes = kBN * kHD * 2;    // 16 KB per stage
constexpr int kTmemCols = 512;        // per lane 256: S/P double buffer [0,64) [64,128), O [128,256)
constexpr int kCh = 16;               // keys per softmax chunk
constexpr float kLog2eT = 1.4426950408889634f;
constexpr float kLn2T = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;

__device__ __forceinline__ void tmem_ldc(uint32_t a, uint32_t (&r)[16]) { tmem_ld16(a, r); }
__device__ __forceinline__ void tmem_stc(uint32_t a, const uint32_t (&r)[8]) { tmem_st8(a, r); }
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __host__ __forceinline__ int q_box_sel(int n_rows) { return n_rows <= 32 ? 0 : (n_rows <= 64 ? 1 : 2); }
__device__ __host__ __forceinline__ int kv_box_sel(int n_valid) { return n_valid <= 32 ? 0 : 1; }

struct PairParams {
    CUtensorMap mq[3], mk[2], mv[2];  // box rows: Q 32 / 64 / 128, K and V 32 / 64
    const TcHeader *hdr;
    const TcTile *tiles;
    const PairRec *pairs;
    uint32_t *status;
    __nv_bfloat16 *out;
    float *lse;
    int n_heads, kv_group;
    int64_t total_tokens;
    float scale_log2e;
    const float *pos, *slopes;        // ALiBi variant
    int stall_producer;               // test hook
};

struct KvTile {
    int row0, n_valid, k_off;
};

// A lane's own view of the work: the items in which it has a tile, and inside an item the key
// tiles that tile reads (all of the preamble's, then the segment's own up to its diagonal).
// g counts the lane's key tiles (parity of its S/P buffers), item_no its items.
struct LaneCursor {
    const TcTile *tiles;
    const PairRec *pairs;
    uint32_t it, n_items, stride, g, item_no;
    int n_heads, lane_id, h, j, n_kv, n_pre;
    TcTile t;
    bool valid;
    __device__ __forceinline__ void load()
    {
        valid = false;
        while (it < n_items) {
            const uint32_t pi = it / (uint32_t)n_heads;
            const PairRec pr = pairs[pi];
            if (lane_id < pr.n) {
                h = (int)(it - pi * (uint32_t)n_heads);
                t = tiles[pr.tile0 + lane_id];
                n_pre = (t.pre_len + kBN - 1) / kBN;
                n_kv = n_pre + (t.q_off + t.n_rows + kBN - 1) / kBN;
                j = 0;
                valid = true;
                return;
            }
            it += stride;
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
    __device__ __forceinline__ void init(const TcTile *tl, const PairRec *pr, uint32_t n, int heads, int lane)
    {
        tiles = tl; pairs = pr; n_items = n; n_heads = heads; lane_id = lane;
        it = blockIdx.x; stride = gridDim.x; g = 0; item_no = 0;
        load();
    }
    __device__ __forceinline__ void next_item() { it += stride; ++item_no; load(); }
    __device__ __forceinline__ void next()
    {
        ++g;
        if (++j == n_kv) next_item();
    }
    __device__ __forceinline__ bool last_of_item() const { return j == n_kv - 1; }
};

// The ring's view: every key tile the block loads, in load order.  r counts stages since the
// block started: slot r % kNS, fill r / kNS (barrier parity (r / kNS) & 1).
struct RingCursor {
    const TcTile *tiles;
    const PairRec *pairs;
    uint32_t it, n_items, stride, r, item_no0, item_no1;
    int n_heads, h, n, j, n_pre, n_own0, n_own1, n_st, own_keys;
    int pre_row, pre_len, own_row, q_row0, q_row1, n_rows0, n_rows1;
    bool valid;
    __device__ __forceinline__ void load()
    {
        valid = it < n_items;
        if (valid) {
            const uint32_t pi = it / (uint32_t)n_heads;
            const PairRec pr = pairs[pi];
            h = (int)(it - pi * (uint32_t)n_heads);
            n = pr.n;
            const TcTile t0 = tiles[pr.tile0];
            pre_row = t0.pre_row; pre_len = t0.pre_len; own_row = t0.own_row; q_row0 = t0.q_row; n_rows0 = t0.n_rows;
            n_pre = (t0.pre_len + kBN - 1) / kBN;
            own_keys = t0.q_off + t0.n_rows;
            n_own0 = (own_keys + kBN - 1) / kBN;
            n_own1 = 0; q_row1 = 0; n_rows1 = 0;
            if (n == 2) {
                const TcTile t1 = tiles[pr.tile0 + 1];
                q_row1 = t1.q_row; n_rows1 = t1.n_rows;
                own_keys = t1.q_off + t1.n_rows;
                n_own1 = (own_keys + kBN - 1) / kBN;
            }
            n_st = n_pre + max(n_own0, n_own1);
            j = 0;
        }
    }
    __device__ __forceinline__ void init(const TcTile *tl, const PairRec *pr, uint32_t nn, int heads)
    {
        tiles = tl; pairs = pr; n_items = nn; n_heads = heads; it = blockIdx.x; stride = gridDim.x; r = 0;
        item_no0 = item_no1 = 0;
        load();
    }
    __device__ __forceinline__ KvTile kv() const
    {
        KvTile k;
        if (j < n_pre) {
            k.row0 = pre_row + j * kBN; k.n_valid = min(kBN, pre_len - j * kBN); k.k_off = -1;
        } else {
            const int o = (j - n_pre) * kBN;
            k.row0 = own_row + o; k.n_valid = min(kBN, own_keys - o); k.k_off = o;
        }
        return k;
    }
    // does lane L multiply with the current stage / is it the first, the last stage of L's item
    __device__ __forceinline__ bool mine(int L) const { return L == 0 ? j < n_pre + n_own0 : (n == 2 && j < n_pre + n_own1); }
    __device__ __forceinline__ bool first(int L) const { return j == 0 && L < n; }
    __device__ __forceinline__ bool last(int L) const { return L < n && j == n_pre + (L == 0 ? n_own0 : n_own1) - 1; }
    __device__ __forceinline__ uint32_t item_no(int L) const { return L == 0 ? item_no0 : item_no1; }
    __device__ __forceinline__ int q_row(int L) const { return L == 0 ? q_row0 : q_row1; }
    __device__ __forceinline__ int n_rows(int L) const { return L == 0 ? n_rows0 : n_rows1; }
    __device__ __forceinline__ uint32_t slot() const { return r % kNS; }
    __device__ __forceinline__ uint32_t parity() const { return (r / kNS) & 1; }
    __device__ __forceinline__ void next()
    {
        ++r;
        if (++j == n_st) { item_no0 += 1; item_no1 += (n == 2); it += stride; load(); }
    }
};

// Shared ring barriers, then one set per lane.
enum { RB_K_FULL = 0, RB_V_FULL = RB_K_FULL + kNS, RB_K_FREE = RB_V_FULL + kNS, RB_V_FREE = RB_K_FREE + kNS,
       RB_V_CLEAN = RB_V_FREE + kNS, RB_COUNT = RB_V_CLEAN + kNS };
enum { BAR_Q_FULL = 0, BAR_Q_EMPTY, BAR_S_FULL, BAR_P_FULL = BAR_S_FULL + 2, BAR_O_DONE = BAR_P_FULL + 2,
       BAR_L_READY = BAR_O_DONE + 2, BAR_X_FREE = BAR_L_READY + 2, BAR_O_FREE = BAR_X_FREE + 2, BAR_DRAIN, BAR_COUNT };

template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

template <bool ALIBI>
__global__ void __launch_bounds__(kThreads, 1) prefill_pair_kernel(const __grid_constant__ PairParams p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char *sQ0 = smem;                                  // [2 lanes] 128 rows x 128 cols, two 64-col halves
    unsigned char *sK = smem + 2 * kQBytes;                     // [kNS] 64 keys x 128 cols
    unsigned char *sV = sK + kNS * kKVBytes;                    // [kNS]
    unsigned char *sO = sV + kNS * kKVBytes;                    // [2 lanes][4 warps] 32 rows x 64 bytes, output staging
    __shared__ uint64_t ring[RB_COUNT];
    __shared__ uint64_t lane_bars[2][BAR_COUNT];
    __shared__ uint32_t tmem_base_s;
    __shared__ float x_l[2][2][kBM];                            // [lane][item parity][row] row sums
    __shared__ float x_m[2][2][kBM];                            // reference maxima

    const int warp_all = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int L = warp_all / kLaneWarps;                        // which tile of the pair this warp serves
    const int warp = warp_all - L * kLaneWarps;                 // role index inside the lane
    uint64_t *lb = lane_bars[L];
    unsigned char *sQ = sQ0 + L * kQBytes;
    if (threadIdx.x == 0) {
        for (int i = 0; i < RB_COUNT; ++i) mbar_init(&ring[i], (i >= RB_K_FREE && i < RB_V_FREE) ? 2 : ((i >= RB_V_FREE && i < RB_V_CLEAN) ? 3 : 1));
        for (int l2 = 0; l2 < 2; ++l2)
            for (int i = 0; i < BAR_COUNT; ++i)
                mbar_init(&lane_bars[l2][i], ((i >= BAR_P_FULL && i < BAR_P_FULL + 2) || (i >= BAR_L_READY && i <= BAR_O_FREE)) ? 128 : 1);
        fence_mbar_init();
        for (int i = 0; i < 3; ++i) prefetch_tmap(&p.mq[i]);
        for (int i = 0; i < 2; ++i) { prefetch_tmap(&p.mk[i]); prefetch_tmap(&p.mv[i]); }
    }
    if (warp_all == 9) { tmem_alloc(&tmem_base_s, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base_s + (uint32_t)L * 256u;       // this lane's S0 [0,64) S1 [64,128) O [128,256)
    const uint32_t n_items = p.hdr->n_pairs * (uint32_t)p.n_heads;
    bool ok = true;

    if (warp >= 8) {
        reg_dealloc<72>();
        if (warp == 8 && L == 0) {
            // -------------------------------------------------------------- TMA producer (both lanes)
            if (lane == 0) {
                uint32_t nq0 = 0, nq1 = 0, n_k = 0, n_v = 0;      // loads issued (Q per lane; K and V stages)
                RingCursor c;
#pragma unroll 1
                for (c.init(p.tiles, p.pairs, n_items, p.n_heads); c.valid && ok && !p.stall_producer; c.next()) {
                    const int hk = c.h / p.kv_group;
                    if (c.j == 0) {
                        for (int l2 = 0; l2 < c.n && ok; ++l2) {
                            if (!(ok = mbar_wait(&lane_bars[l2][BAR_Q_EMPTY], (c.item_no(l2) & 1) ^ 1))) break;
                            const int qs = q_box_sel(c.n_rows(l2));
                            mbar_expect_tx(&lane_bars[l2][BAR_Q_FULL], (32u << qs) * (kHD * 2));
                            tma_load_3d(sQ0 + l2 * kQBytes, &p.mq[qs], 0, c.q_row(l2), c.h * 2, &lane_bars[l2][BAR_Q_FULL]);
                            if (l2 == 0) ++nq0; else ++nq1;
                        }
                        if (!ok) break;
                    }
                    const KvTile kt = c.kv();
                    const uint32_t sl = c.slot(), ph = c.parity();
                    if (c.r >= kNS && !(ok = mbar_wait(&ring[RB_K_FREE + sl], ph ^ 1))) break;
                    const int ks = kv_box_sel(kt.n_valid);
                    mbar_expect_tx(&ring[RB_K_FULL + sl], (32u << ks) * (kHD * 2));
                    tma_load_3d(sK + sl * kKVBytes, &p.mk[ks], 0, kt.row0, hk * 2, &ring[RB_K_FULL + sl]);
                    ++n_k;
                    if (c.r >= kNS && !(ok = mbar_wait(&ring[RB_V_FREE + sl], ph ^ 1))) break;
                    mbar_expect_tx(&ring[RB_V_FULL + sl], (32u << ks) * (kHD * 2));
                    tma_load_3d(sV + sl * kKVBytes, &p.mv[ks], 0, kt.row0, hk * 2, &ring[RB_V_FULL + sl]);
                    ++n_v;
                }
                if (!ok) {
                    // a wait ran out: before the block may exit, its own copies in flight must have landed
                    if (nq0) mbar_wait(&lane_bars[0][BAR_Q_FULL], (nq0 - 1) & 1);
                    if (nq1) mbar_wait(&lane_bars[1][BAR_Q_FULL], (nq1 - 1) & 1);
                    for (uint32_t sl = 0; sl < kNS; ++sl) {      // the last fill of every slot that was ever filled
                        if (n_k > sl) mbar_wait(&ring[RB_K_FULL + sl], (((n_k - 1 - sl) / kNS)) & 1);
                        if (n_v > sl) mbar_wait(&ring[RB_V_FULL + sl], (((n_v - 1 - sl) / kNS)) & 1);
                    }
                }
            }
        } else if (warp == 9) {
            // -------------------------------------------------------------- MMA issuer of this lane
            if (lane == 0) {
                const uint32_t d_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
                const uint32_t q_lo = ((smem_u32(sQ) & 0x3ffffu) >> 4) | (1u << 16);
                const uint32_t k_lo = ((smem_u32(sK) & 0x3ffffu) >> 4) | (1u << 16);
                const uint32_t v_lo = (smem_u32(sV) & 0x3ffffu) >> 4;
                const uint32_t id_o = idesc_bf16(kBM, kHD, 0, 1);
                uint32_t rag = 0;                   // bit sl: parity of the ragged stages seen in slot sl (phase of V_CLEAN)
                // cs: next stage whose S = Q K^T may be issued; cp: next stage whose O += P V may be issued.
                // Stages the lane does not multiply with are skipped here (its pass-by thread releases them).
                // gs / gp: the lane's own tiles issued so far on either side; S runs at most two ahead.
                RingCursor cs, cp;
                cs.init(p.tiles, p.pairs, n_items, p.n_heads);
                cp.init(p.tiles, p.pairs, n_items, p.n_heads);
                uint32_t gs = 0, gp = 0;
                // Every stage is waited for in ring order on both sides, also the ones this lane does not
                // multiply with: a thread that skipped them could be two fills ahead of a slot's barrier,
                // where a parity wait answers for the wrong fill.
                uint64_t idle_since = 0;            // start of the current stretch without any progress (0: none)
#pragma unroll 1
                while (ok && (cs.valid || cp.valid)) {
                    const uint32_t mark = cs.r + cp.r + gs + gp;
                    // ---- S side: as far as operands have landed; at most two of the lane's tiles ahead
#pragma unroll 1
                    while (cs.valid) {
                        const uint32_t sl = cs.slot();
                        if (!cs.mine(L)) {               // not this lane's: release it once its load has landed
                            if (!mbar_test(&ring[RB_K_FULL + sl], cs.parity())) break;
                            mbar_arrive(&ring[RB_K_FREE + sl]);
                            cs.next();
                            continue;
                        }
                        if (gs >= gp + 2) break;
                        const bool first = cs.first(L);
                        const bool ready = mbar_test(&ring[RB_K_FULL + sl], cs.parity()) &&
                                           (!first || mbar_test(&lb[BAR_Q_FULL], cs.item_no(L) & 1));
                        if (!ready && gs != gp) break;          // look-ahead only when nothing has to be waited for
                        if (first && !(ok = mbar_wait(&lb[BAR_Q_FULL], cs.item_no(L) & 1))) break;
                        if (!(ok = mbar_wait(&ring[RB_K_FULL + sl], cs.parity()))) break;
                        tc_fence_after();
                        const uint32_t st = gs & 1;
                        const int n_valid = cs.kv().n_valid;
                        const int n_mma = (n_valid + 15) & ~15;
                        const uint32_t id_s = idesc_bf16(kBM, 0, 0, 0) | ((uint32_t)(n_mma >> 3) << 17);
                        const uint32_t kb = k_lo + sl * (kKVBytes >> 4);
                        const uint32_t d = tb + st * kBN;
                        const uint32_t q_half = (32u << q_box_sel(cs.n_rows(L))) * 8u;
                        const uint32_t k_half = (32u << kv_box_sel(n_valid)) * 8u;
#pragma unroll
                        for (int kk = 0; kk < kHD / 16; ++kk)
                            umma_ss_lh(d, q_lo + (kk >> 2) * q_half + (kk & 3) * 2,
                                       kb + (kk >> 2) * k_half + (kk & 3) * 2, d_hi, id_s, kk > 0 ? 1u : 0u);
                        umma_commit(&lb[BAR_S_FULL + st]);
                        umma_commit(&ring[RB_K_FREE + sl]);
                        if (cs.last(L)) umma_commit(&lb[BAR_Q_EMPTY]);
                        ++gs;
                        cs.next();
                    }
                    if (ok && cp.valid && !(cp.mine(L) && gp == gs)) idle_since = 0;     // the O += P V side below makes progress or waits with its own limit
                    else if (ok && mark == cs.r + cp.r + gs + gp) {                      // nothing moved: polling, with the same limit as every wait
                        const uint64_t now = global_timer_ns();
                        if (idle_since == 0) idle_since = now;
                        else if (now - idle_since > kWaitLimitNs) { ok = false; break; }
                    } else idle_since = 0;
                    if (!ok || !cp.valid) continue;
                    // ---- O += P V side: one stage
                    const uint32_t sl = cp.slot();
                    const int pv_valid = cp.kv().n_valid;
                    if (!cp.mine(L)) {
                        if (!(ok = mbar_wait(&ring[RB_V_FULL + sl], cp.parity()))) break;
                        mbar_arrive(&ring[RB_V_FREE + sl]);
                        if (pv_valid & 15) rag ^= 1u << sl;
                        cp.next();
                        continue;
                    }
                    if (gp == gs) continue;                     // its S = Q K^T is not issued yet: back to the S side
                    const uint32_t st = gp & 1, ph = (gp >> 1) & 1;
                    const int n_k = (pv_valid + 15) >> 4;
                    if (!(ok = mbar_wait(&lb[BAR_P_FULL + st], ph))) break;
                    if (!(ok = mbar_wait(&ring[RB_V_FULL + sl], cp.parity()))) break;
                    if (pv_valid & 15) {
                        const uint32_t par = (rag >> sl) & 1;
                        rag ^= 1u << sl;
                        if (!(ok = mbar_wait(&ring[RB_V_CLEAN + sl], par))) break;
                    }
                    const bool first = cp.first(L);
                    if (first && cp.item_no(L) > 0 && !(ok = mbar_wait(&lb[BAR_O_FREE], (cp.item_no(L) - 1) & 1))) break;
                    tc_fence_after();
                    const uint32_t vb = (v_lo + sl * (kKVBytes >> 4)) | (((32u << kv_box_sel(pv_valid)) * 8u) << 16);
                    const uint32_t pa = tb + st * kBN;
#pragma unroll
                    for (int kk = 0; kk < kBN / 16; ++kk)
                        if (kk < n_k)
                            umma_ts_lh(tb + 128, pa + kk * 8, vb + kk * (2048 >> 4), d_hi, id_o, (!first || kk > 0) ? 1u : 0u);
                    umma_commit(&lb[BAR_O_DONE + st]);
                    umma_commit(&ring[RB_V_FREE + sl]);
                    ++gp;
                    cp.next();
                }
                if (!ok) {
                    umma_commit(&lb[BAR_DRAIN]);
                    mbar_wait(&lb[BAR_DRAIN], 0);
                }
            }
        } else if (warp == 10 && L == 0) {
            // -------------------------------------------------------------- V cleaner (all stages)
            RingCursor c;
#pragma unroll 1
            for (c.init(p.tiles, p.pairs, n_items, p.n_heads); c.valid && ok; c.next()) {
                const int n_valid = c.kv().n_valid;
                const uint32_t sl = c.slot();
                if (!(ok = mbar_wait_warp(&ring[RB_V_FULL + sl], c.parity()))) break;
                // the cleaner is the third party every V stage is released by: it waits on every fill, so it
                // must not be able to fall a whole fill behind the ring
                if ((n_valid & 15) == 0) {
                    if (lane == 0) mbar_arrive(&ring[RB_V_FREE + sl]);
                    continue;
                }
                const int n_mma = (n_valid + 15) & ~15;
                const int half_bytes = (32 << kv_box_sel(n_valid)) * 128;
                unsigned char *vs = sV + sl * kKVBytes;
                for (int i = lane; i < (n_mma - n_valid) * 16; i += 32) {
                    const int rr = n_valid + (i >> 4), half = (i >> 3) & 1, piece = i & 7;
                    *reinterpret_cast<uint4 *>(vs + half * half_bytes + rr * 128 + piece * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&ring[RB_V_CLEAN + sl]); mbar_arrive(&ring[RB_V_FREE + sl]); }
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        // ------------------------------------------------------------------ softmax (one thread per query row)
        reg_alloc<88>();
        const int row = warp * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const float sc = p.scale_log2e;
        LaneCursor c;
        c.init(p.tiles, p.pairs, n_items, p.n_heads, L);
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
            if (!(ok = mbar_wait_warp(&lb[BAR_S_FULL + st], (c.g >> 1) & 1))) break;
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
                }
                // keys past the row's limit (causal diagonal, ragged tail) -> -inf; skipped when the
                // whole warp sees the whole chunk
                if (ch * kCh + 16 > lim0) {
#pragma unroll
                    for (int i = 0; i < kCh; ++i) r[i] = (ch * kCh + i < lim) ? r[i] : 0xff800000u;
                }
#pragma unroll
                for (int i = 0; i < kCh; ++i) mx[i & 3] = fmaxf(mx[i & 3], __uint_as_float(r[i]));
            }
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
                if (!(ok = mbar_wait_warp(&lb[BAR_O_DONE + ((c.g - 1) & 1)], ((c.g - 1) >> 1) & 1))) break;
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
                float rs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
                for (int ch = 0; ch < n_ch; ++ch) {     // pass 2: P = exp2(score - reference) as bf16, written over S
                    uint32_t pk[kCh / 2];
                    if (ch < see) {
                        uint32_t r[kCh];
                        tmem_ldc(s_addr + ch * kCh, r);
                        tmem_ld_wait();
                        if (ALIBI) {
                            const float kp = ch < 2 ? kp0 : kp1;
#pragma unroll
                            for (int i = 0; i < kCh; ++i) {
                                const float pkey = __shfl_sync(0xffffffffu, kp, (ch & 1) * kCh + i);
                                r[i] = __float_as_uint(fmaf(__uint_as_float(r[i]), sc, -slope_l2 * fabsf(pq - pkey)));
                            }
                        }
                        if (ch * kCh + 16 > lim0) {
#pragma unroll
                            for (int i = 0; i < kCh; ++i) r[i] = (ch * kCh + i < lim) ? r[i] : 0xff800000u;
                        }
#pragma unroll
                        for (int i = 0; i < kCh; i += 2) {
                            const float p0 = ex2(fmaf(__uint_as_float(r[i]), sc_exp, nm));
                            const float p1 = ex2(fmaf(__uint_as_float(r[i + 1]), sc_exp, nm));
                            rs[(i >> 1) & 3] += p0 + p1;
                            pk[i >> 1] = pack_bf16x2(p0, p1);
                        }
                    } else {                            // keys no row of this warp sees
#pragma unroll
                        for (int i = 0; i < kCh / 2; ++i) pk[i] = 0u;
                    }
                    // P chunk ch (8 columns of bf16 pairs) lands on score columns already consumed
                    tmem_stc(s_addr + ch * (kCh / 2), pk);
                }
                l += (rs[0] + rs[1]) + (rs[2] + rs[3]);
            }
            // P of this tile is in TMEM: release the tile to the MMA issuer
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&lb[BAR_P_FULL + st]);
            if (c.last_of_item()) {                 // hand the item's row statistics to the epilogue warps
                const uint32_t xp = c.item_no & 1;
                // the slot was last used two items ago: the epilogue must have read it
                if (c.item_no >= 2 && !(ok = mbar_wait_warp(&lb[BAR_X_FREE + xp], ((c.item_no >> 1) - 1) & 1))) break;
                x_l[L][xp][row] = l;
                x_m[L][xp][row] = m_ref;
                mbar_arrive(&lb[BAR_L_READY + xp]);
            }
            c.next();
        }
    } else {
        // ------------------------------------------------------------------ epilogue of this lane (warps 4-7 of it)
        // O / l -> bf16 -> global and the log-sum-exp, off the softmax warps' critical path.
        const int quad = warp - 4;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        unsigned char *stage = sO + L * 8192 + quad * 2048;
        const int64_t row_pitch = (int64_t)p.n_heads * kHD * 2;
        uint32_t g_end = 0;
        LaneCursor c;
#pragma unroll 1
        for (c.init(p.tiles, p.pairs, n_items, p.n_heads, L); c.valid && ok; c.next_item()) {
            const TcTile t = c.t;
            const int h = c.h;
            const uint32_t item_no = c.item_no;
            g_end += (uint32_t)c.n_kv;
            const uint32_t g_last = g_end - 1;
            const int xp = item_no & 1;
            if (!(ok = mbar_wait_warp(&lb[BAR_L_READY + xp], (item_no >> 1) & 1))) break;
            const float l_row = x_l[L][xp][row], m_row = x_m[L][xp][row];
            mbar_arrive(&lb[BAR_X_FREE + xp]);
            if (!(ok = mbar_wait_warp(&lb[BAR_O_DONE + (g_last & 1)], (g_last >> 1) & 1))) break;   // last O += P V
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
                    mbar_arrive(&lb[BAR_O_FREE]);
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
                        if (quad * 32 + rr < t.n_rows)
                            *reinterpret_cast<uint4 *>(dst + (int64_t)(quad * 32 + rr) * row_pitch + cc * 64 + piece * 16) = w;
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
    if (warp_all == 9) tmem_dealloc(tmem_base_s, kTmemCols);
}

}  // namespace pair

// ---- host side ---------------------------------------------------------------------------
int make_rows_tensor_map(CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int box_rows);   // prefill_tc.cu
bool prefill_stall_hook();                                                                               // prefill_tc.cu

int launch_prefill_pair(const void *q, const void *k, const void *v, const sp_layout *lay, const float *pos,
                        const float *slopes, int n_heads, int n_kv_heads, float scale, void *out, float *lse,
                        void *ws, cudaStream_t st)
{
    using namespace pair;
    PairParams p;
    for (int i = 0; i < 3; ++i)
        if (int rc = make_rows_tensor_map(&p.mq[i], q, lay->total_tokens, (int64_t)n_heads * kHD, 32 << i)) return rc;
    for (int i = 0; i < 2; ++i) {
        if (int rc = make_rows_tensor_map(&p.mk[i], k, lay->total_tokens, (int64_t)n_kv_heads * kHD, 32 << i)) return rc;
        if (int rc = make_rows_tensor_map(&p.mv[i], v, lay->total_tokens, (int64_t)n_kv_heads * kHD, 32 << i)) return rc;
    }
    const int64_t cap = plan_max_tiles(lay->n_prompts, lay->n_paths, lay->max_pre_len, lay->max_path_len, kBM);
    TcHeader *hdr = static_cast<TcHeader *>(ws);
    TcTile *tiles = reinterpret_cast<TcTile *>(static_cast<char *>(ws) + 256);
    PairRec *pairs = reinterpret_cast<PairRec *>(static_cast<char *>(ws) + 256 + round_up((size_t)cap * sizeof(TcTile), 256));
    SP_CUDA(cudaMemsetAsync(ws, 0, 256, st));

    PlanArgs pa;
    pa.ppo = lay->prompt_path_off; pa.pre_start = lay->pre_start; pa.pre_len = lay->pre_len;
    pa.path_start = lay->path_start; pa.doc_len = lay->doc_len; pa.qry_len = lay->qry_len;
    pa.n_prompts = lay->n_prompts; pa.n_paths = lay->n_paths; pa.rows_mode = SP_ROWS_ALL; pa.tile_rows = kBM;
    pa.max_pre_len = lay->max_pre_len; pa.max_path_len = lay->max_path_len; pa.total_tokens = lay->total_tokens;
    pa.max_tiles = cap;
    pa.hdr = hdr; pa.tiles = tiles; pa.pairs = pairs;
    prefill_plan_kernel<<<1, 1024, 0, st>>>(pa);
    SP_CUDA(cudaGetLastError());

    p.hdr = hdr; p.tiles = tiles; p.pairs = pairs; p.status = &hdr->status;
    p.out = static_cast<__nv_bfloat16 *>(out); p.lse = lse;
    p.n_heads = n_heads; p.kv_group = n_heads / n_kv_heads;
    p.total_tokens = lay->total_tokens; p.scale_log2e = scale * kLog2eT;
    p.pos = pos; p.slopes = slopes;
    p.stall_producer = prefill_stall_hook() ? 1 : 0;

    const int64_t items = cap * n_heads;             // upper bound on pairs x heads
    if (items == 0) return SP_OK;
    const int grid = (int)std::min<int64_t>(items, num_sms());
    const int smem = 2 * kQBytes + 2 * kNS * kKVBytes + 2 * 4 * 2048 + 1024;
    if (pos) {
        SP_CUDA(cudaFuncSetAttribute(prefill_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_pair_kernel<true><<<grid, kThreads, smem, st>>>(p);
    } else {
        SP_CUDA(cudaFuncSetAttribute(prefill_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        prefill_pair_kernel<false><<<grid, kThreads, smem, st>>>(p);
    }
    SP_CUDA(cudaGetLastError());
    return SP_OK;
}

}  // namespace sp
