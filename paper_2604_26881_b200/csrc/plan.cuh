// The expert work plan as a device function, so that the small-batch dispatch kernel can build it
// in the same launch.  (Paper Sec. 3 / Sec. 5: G experts per function is the granularity at which
// expert work is partitioned.)
#pragma once

#include "internal.h"
#include "scan.cuh"

namespace faasmoe {

struct PlanArgs {
    const int32_t* slot_table;
    int M, E, G, T, tile_rows;
    const int32_t* model_tok_off;     // null when M == 1
    int with_shared;
    int nblk1, nblk2, snblk1, snblk2; // weight-row blocks of the gate/up and down GEMMs (routed, shared)
    int token_major;                  // 1: units of the one-CTA token-major shape (see the end of plan_body)
    int n_ctas;                       // CTAs of the grouped GEMM launches
    int shared_down_width;            // token-major: weight rows of a shared-expert unit of the down projection
    int split_ok[2];                  // token-major: K / 64 of the routed units is even (gate/up, down)
    int direct;                       // the routed gate/up units read all T tokens in place
    int interleave_down;              // the shared units of the down projection are as long as the routed ones
    Tile* tiles;
    Tile* stiles;
    Unit* units1;                     // null: no unit lists (CUDA-core path)
    Unit* units2;
    int32_t* plan_counts;
};

// Whole block.  expert_off [M*E+1] may live in shared or global memory (already visible to the block).
// s_mem: M*E + M*B + 1 ints of shared memory; s_warp: 33 ints.
__device__ __forceinline__ void plan_body(const int32_t* expert_off, const PlanArgs& a, int32_t* s_mem, int32_t* s_warp)
{
    const int ME = a.M * a.E;
    const int B = (a.E + a.G - 1) / a.G;
    const int NG = a.M * B;
    int32_t* s_tile_base = s_mem;            // [ME]   tiles before expert i
    int32_t* s_group_tile0 = s_mem + ME;     // [NG+1] first tile of each expert block
    const int tid = threadIdx.x, nth = blockDim.x;

    for (int i = tid; i < ME; i += nth) {
        const int cnt = expert_off[i + 1] - expert_off[i];
        s_tile_base[i] = (cnt + a.tile_rows - 1) / a.tile_rows;
    }
    __syncthreads();
    const int n_tiles = block_scan_exclusive(s_tile_base, ME, s_warp);
    for (int i = tid; i < ME; i += nth) {
        const int m = i / a.E, e = i - m * a.E;
        const int row_begin = expert_off[i], row_end = expert_off[i + 1];
        int tix = s_tile_base[i];
        for (int r = row_begin; r < row_end; r += a.tile_rows, ++tix) {
            Tile t;
            t.row0 = r;
            t.nrows = min(a.tile_rows, row_end - r);
            t.slot = a.slot_table[i];
            t.group = m * B + e / a.G;
            a.tiles[tix] = t;
        }
    }
    for (int gidx = tid; gidx <= NG; gidx += nth) {
        int v = n_tiles;
        if (gidx < NG) {
            const int m = gidx / B, b = gidx - m * B;
            v = s_tile_base[m * a.E + b * a.G];
        }
        s_group_tile0[gidx] = v;
    }
    __syncthreads();

    // shared-expert tiles: tokens of one model, tile_rows at a time
    int n_stiles = 0;
    if (a.with_shared) {
        for (int m = 0; m < a.M; ++m) {
            const int t_begin = a.model_tok_off ? a.model_tok_off[m] : 0;
            const int t_end = a.model_tok_off ? a.model_tok_off[m + 1] : a.T;
            const int nt = (t_end - t_begin + a.tile_rows - 1) / a.tile_rows;
            for (int i = tid; i < nt; i += nth) {
                Tile t;
                t.row0 = t_begin + i * a.tile_rows;
                t.nrows = min(a.tile_rows, t_end - t.row0);
                t.slot = m;
                t.group = m;
                a.stiles[n_stiles + i] = t;
            }
            n_stiles += nt;
        }
    }

    // Unit lists of the grouped GEMMs.  Shared-expert units come first (the longest ones of the down
    // projection), then the routed units ordered by (expert block, weight-row block, tile): all
    // experts of a block advance through the same weight-row block together.
    if (a.units1) {
        const int su1 = n_stiles * a.snblk1, su2 = n_stiles * a.snblk2;
        // Token-major units: the colblock is (first weight row / 64) with a width code in the top byte (0: 256 weight
        // rows, 1: 128, 2: 64); narrower units pack 2 or 4 K slices into a stage, so a unit of half the rows is half
        // as long.  The shared expert's down projection contracts over 4x more elements than a routed expert's; with
        // few tokens its units are made 4x (2x) narrower so that they are as long as the routed ones.
        const int tm = a.token_major;
        const int wsh = a.shared_down_width;
        const int sh_step = wsh / 64, sh_code = wsh == 256 ? 0 : (wsh == 128 ? 1 : 2);
        for (int i = tid; i < su1; i += nth) { Unit u; u.colblock = (i / n_stiles) * (tm ? 4 : 1); u.tile = ~(i % n_stiles); a.units1[i] = u; }
        for (int i = tid; i < su2; i += nth) {
            Unit u;
            const int cb = i / n_stiles;
            u.colblock = tm ? (cb * sh_step) | (sh_code << 24) : cb;
            u.tile = ~(i % n_stiles);
            a.units2[i] = u;
        }
        const int nmax = n_tiles * max(a.nblk1, a.nblk2);
        for (int i = tid; i < nmax; i += nth) {
            const int tile = i % n_tiles, cb = i / n_tiles;
            // expert block of the tile: last block whose first tile is <= tile
            int lo = 0, hi = NG;
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_group_tile0[mid] <= tile) lo = mid; else hi = mid; }
            // empty blocks share their first tile with the next one: step to the last of them
            const int t0 = s_group_tile0[lo], nt = s_group_tile0[lo + 1] - t0;
            Unit u; u.colblock = cb * (tm ? 4 : 1); u.tile = tile;
            if (cb < a.nblk1) a.units1[su1 + t0 * a.nblk1 + cb * nt + (tile - t0)] = u;
            if (cb < a.nblk2) a.units2[su2 + t0 * a.nblk2 + cb * nt + (tile - t0)] = u;
        }
        if (tid == 0) {
            a.plan_counts[2] = su1 + n_tiles * a.nblk1;
            a.plan_counts[3] = su2 + n_tiles * a.nblk2;
            // shared units that the scheduler spreads over the launch: only where a model's tokens fill several tiles
            // (its shared weights are then read again and again out of L2, while a single tile streams them from HBM
            // like any routed expert), and only equally long units (longer ones go first)
            const bool reread = n_stiles > a.M;
            a.plan_counts[6] = reread ? su1 : 0;
            a.plan_counts[7] = (reread && a.interleave_down) ? su2 : 0;
        }
        if (a.token_major) {
            // U equally long units on S CTAs take ceil(U / S) rounds; when the last round is less than half full, its
            // units (the tail of the list: routed ones) are split into two units of half the weight rows each, where
            // the tile has at most 64 rows, so that round costs half.
            __shared__ int s_split[128];
            int r2[2];
            for (int l = 0; l < 2; ++l) {
                const int routed = n_tiles * (l ? a.nblk2 : a.nblk1);
                const int total = (l ? su2 : su1) + routed;
                int r = total % a.n_ctas;
                if (2 * r > a.n_ctas || r > routed || r > 128 || !a.split_ok[l]) r = 0;
                r2[l] = r;
            }
            for (int l = 0; l < 2; ++l) {
                const int r = r2[l];
                if (r == 0) continue;                                       // (the same decision in every thread)
                Unit* list = l ? a.units2 : a.units1;
                const int total = (l ? su2 : su1) + n_tiles * (l ? a.nblk2 : a.nblk1);
                __syncthreads();                                            // the list is complete
                Unit mine;
                int cnt = 0;
                if (tid < r) {
                    mine = list[total - r + tid];
                    const int rows = a.direct ? a.T : a.tiles[mine.tile].nrows;
                    cnt = rows <= 64 ? 2 : 1;
                }
                // position of each unit after the split: a prefix count of the units that become two (r <= 128: the
                // first four warps hold them all)
                const unsigned two = __ballot_sync(0xffffffffu, cnt == 2);
                if (tid < 128 && (tid & 31) == 0) s_split[tid >> 5] = __popc(two);
                __syncthreads();
                if (tid < r) {
                    int off = tid + __popc(two & ((1u << (tid & 31)) - 1u));
                    for (int w = 0; w < (tid >> 5); ++w) off += s_split[w];
                    Unit u = mine;
                    if (cnt == 2) {
                        u.colblock = mine.colblock | (1 << 24);
                        list[total - r + off] = u;
                        u.colblock = (mine.colblock + 2) | (1 << 24);
                        list[total - r + off + 1] = u;
                    } else {
                        list[total - r + off] = u;
                    }
                }
                if (tid == 0) a.plan_counts[2 + l] = total + s_split[0] + s_split[1] + s_split[2] + s_split[3];
                __syncthreads();
            }
        }
    }
    if (tid == 0) {
        a.plan_counts[0] = n_tiles;
        a.plan_counts[1] = n_stiles;
        a.plan_counts[4] = 0;           // work counters of the two grouped GEMM launches
        a.plan_counts[5] = 0;
    }
}

}  // namespace faasmoe
