// Tile list shared by the tensor-core prefill kernels: a one-block plan kernel turns the ragged
// fork-join layout (Section 3.2) into query tiles of a given height, each knowing its segment,
// its offset inside it and its prompt's fully visible preamble.
#pragma once
#include "common.cuh"

namespace sp {

struct TcTile {                       // one query tile (shared by all heads)
    int32_t q_row;                    // packed row of the tile's first query row
    int32_t n_rows;                   // valid rows in the tile (1..tile height)
    int32_t q_off;                    // offset of the first row inside its segment
    int32_t own_row;                  // packed row of the segment's first row
    int32_t pre_row, pre_len;         // fully visible prefix (the prompt's preamble), may be empty
    int32_t pad0, pad1;
};

struct PairRec {                      // up to two consecutive query tiles of one segment
    int32_t tile0;                    // index of the first one in the tile list
    int32_t n;                        // 1 or 2
};

struct TcHeader {                     // start of the workspace
    uint32_t status;
    uint32_t n_tiles;
    uint32_t n_pairs;
};

// ---- plan: ragged layout -> tile list ---------------------------------------------------
struct PlanArgs {
    const int32_t *ppo, *pre_start, *pre_len, *path_start, *doc_len, *qry_len;
    int n_prompts, n_paths, rows_mode;
    int tile_rows;                    // query rows per tile
    int max_pre_len, max_path_len;    // the host's bounds on the lengths (they sized the tile list)
    int64_t total_tokens;             // T: every segment must lie inside [0, T)
    int64_t max_tiles;                // capacity of the tile list
    TcHeader *hdr;
    TcTile *tiles;
    PairRec *pairs = nullptr;         // optional: the tiles grouped two by two per segment
};

// What the host cannot check, the plan kernel does: a segment whose device-side numbers
// contradict the host scalars (negative or oversized length, rows outside [0, T)) gets no tiles
// and the status word reports it, so nothing outside the caller's tensors is ever touched and
// the tile list cannot outgrow the workspace that was sized from those scalars.

static __global__ void __launch_bounds__(1024) prefill_plan_kernel(const PlanArgs a)
{
    __shared__ int warp_tot[32], warp_tot2[32];
    __shared__ int running, running2;
    if (threadIdx.x == 0) { running = 0; running2 = 0; }
    __syncthreads();
    const int n_seq = a.n_prompts + a.n_paths;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < n_seq; base += 1024) {
        const int s = base + threadIdx.x;
        int first = 0, rows = 0, own_row = 0, pre_row = 0, pre_n = 0;
        bool bad = false;
        if (s < a.n_prompts) {
            const int len = a.pre_len[s], row = a.pre_start[s];
            bad = len < 0 || len > a.max_pre_len || row < 0 || (int64_t)row + len > a.total_tokens;
            if (a.rows_mode == SP_ROWS_ALL && !bad) { rows = len; own_row = row; }
        } else if (s < n_seq) {
            const int i = s - a.n_prompts;
            int lo = 0, hi = a.n_prompts - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (a.ppo[mid] <= i) lo = mid; else hi = mid - 1;
            }
            pre_row = a.pre_start[lo]; pre_n = a.pre_len[lo];
            own_row = a.path_start[i];
            const int dl = a.doc_len[i], ql = a.qry_len[i];
            bad = dl < 0 || ql < 0 || (int64_t)dl + ql > a.max_path_len || own_row < 0 ||
                  (int64_t)own_row + dl + ql > a.total_tokens ||
                  pre_n < 0 || pre_n > a.max_pre_len || pre_row < 0 || (int64_t)pre_row + pre_n > a.total_tokens;
#ifdef SP_DEBUG_BOUNDS
            // debug build: no other segment may share a row with this path (every pair is looked at)
            for (int o = 0; o < n_seq && !bad; ++o) {
                if (o == s) continue;
                const int orow = o < a.n_prompts ? a.pre_start[o] : a.path_start[o - a.n_prompts];
                const int olen = o < a.n_prompts ? a.pre_len[o] : a.doc_len[o - a.n_prompts] + a.qry_len[o - a.n_prompts];
                bad = olen > 0 && dl + ql > 0 && orow < own_row + dl + ql && own_row < orow + olen;
            }
#endif
            first = a.rows_mode == SP_ROWS_QUERY_ONLY ? dl : 0;
            rows = bad ? 0 : dl + ql - first;
        }
        if (bad) a.hdr->status = STATUS_BAD_LAYOUT;
        const int nt = (rows + a.tile_rows - 1) / a.tile_rows;
        const int np = (nt + 1) / 2;
        int incl = nt, incl2 = np;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            const int v2 = __shfl_up_sync(0xffffffffu, incl2, o);
            if (lane >= o) { incl += v; incl2 += v2; }
        }
        if (lane == 31) { warp_tot[warp] = incl; warp_tot2[warp] = incl2; }
        __syncthreads();
        int before = running, before2 = running2;
        for (int w = 0; w < warp; ++w) { before += warp_tot[w]; before2 += warp_tot2[w]; }
        int off = before + incl - nt;
        if (a.pairs) {
            const int off2 = before2 + incl2 - np;
            for (int t = 0; t < np && off + 2 * t < a.max_tiles; ++t) {
                PairRec pr;
                pr.tile0 = off + 2 * t;
                pr.n = (2 * t + 1 < nt && off + 2 * t + 1 < a.max_tiles) ? 2 : 1;
                a.pairs[off2 + t] = pr;
            }
        }
        for (int t = 0; t < nt && off + t < a.max_tiles; ++t) {
            TcTile tl;
            tl.q_off = first + t * a.tile_rows;
            tl.q_row = own_row + tl.q_off;
            tl.n_rows = min(a.tile_rows, rows - t * a.tile_rows);
            tl.own_row = own_row;
            tl.pre_row = pre_row; tl.pre_len = pre_n; tl.pad0 = 0; tl.pad1 = 0;
            a.tiles[off + t] = tl;
        }
        __syncthreads();
        if (threadIdx.x == 1023) { running = before + incl; running2 = before2 + incl2; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        a.hdr->n_tiles = (uint32_t)min((int64_t)running, a.max_tiles);
        a.hdr->n_pairs = (uint32_t)min((int64_t)running2, a.max_tiles);
    }
}

static inline int64_t plan_max_tiles(int n_prompts, int n_paths, int max_pre_len, int max_path_len, int tile_rows)
{
    return (int64_t)n_prompts * ((max_pre_len + tile_rows - 1) / tile_rows) +
           (int64_t)n_paths * ((max_path_len + tile_rows - 1) / tile_rows);
}

}  // namespace sp
