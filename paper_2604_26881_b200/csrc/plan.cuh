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
    int split4_ok[2];                 //              ... is divisible by 4
    int direct;                       // the routed gate/up units read all T tokens in place
    int interleave_down;              // the shared units of the down projection are as long as the routed ones
    const int32_t* block_table;       // null: block of expert e = e / G; else [M*E] block ids in [0, table_blocks)
    int table_blocks;
    int short_rows;                   // tiles of at most this many rows are "short" (0: none)
    int32_t* tile_cidx;               // [tiles] rank of a tile among the tiles of its block and class (long / short)
    int private_mode;                 // 1: tiles never span two tenants (private orchestrators batch per tenant)
    const int32_t* bin_off;           //    offsets of the (model, expert, tenant) bins, [nbins + 1]
    const int32_t* bin_base;          //    first bin of each model
    const int32_t* tenants_in_model;
    Tile* tiles;
    Tile* stiles;
    Unit* units1;                     // null: no unit lists (CUDA-core path)
    Unit* units2;
    int32_t* plan_counts;
};

// Whole block.  expert_off [M*E+1] may live in shared or global memory (already visible to the block).
// s_mem: 2*M*E + 2*(M*B + 1) ints of shared memory; s_warp: 33 ints.
__device__ __forceinline__ void plan_body(const int32_t* expert_off, const PlanArgs& a, int32_t* s_mem, int32_t* s_warp)
{
    const int ME = a.M * a.E;
    const int B = a.block_table ? a.table_blocks : (a.E + a.G - 1) / a.G;
    const int NG = a.M * B;
    // block of expert i = (m, e): consecutive experts (Sec. 3: packaged by expert id) or, with a table, any set of
    // experts of the model (load-aware formation, Sec. 5)
    auto block_of = [&](int m, int e) { return m * B + (a.block_table ? a.block_table[m * a.E + e] : e / a.G); };
    int32_t* s_tile_base = s_mem;               // [ME]   tiles before expert i
    int32_t* s_short_base = s_mem + ME;         // [ME]   short tiles before expert i
    int32_t* s_group_long0 = s_mem + 2 * ME;    // [NG+1] long tiles before each expert block
    int32_t* s_group_short0 = s_group_long0 + NG + 1;   // [NG+1] short tiles before each expert block
    const int tid = threadIdx.x, nth = blockDim.x;
    // The common case -- blocks of consecutive experts, no short class -- needs none of the per-block loops and no
    // per-tile lookups below: a block's tiles are consecutive, so every index has a closed form (this kernel sits on the
    // latency chain of small batches).
    const bool simple = a.block_table == nullptr && a.short_rows == 0;
    // Blocks of consecutive experts with a short class, shared orchestrator (large one-model batches): still closed
    // forms -- a block's tiles are consecutive and only the last tile of an expert can be short.
    const bool ranged = a.block_table == nullptr && a.short_rows > 0 && !a.private_mode;
    const bool general = !simple && !ranged;

    // Shared orchestrator (Sec. 4.2): the rows of an expert form one segment whoever owns them, cut into tiles.
    // Private orchestrators: every tenant's rows of an expert are a request of their own, so the segments are the
    // (expert, tenant) bins and no tile spans two tenants.  Row order, and with it every result, is the same.
    // A tile of at most short_rows rows is "short": its units form the tail of the unit lists, from where the
    // background lanes of the pair-shaped grouped GEMM take them (short_rows = 0: no such class).
    for (int i = tid; i < ME; i += nth) {
        const int m = i / a.E, e = i - m * a.E;
        const int tim = a.private_mode ? a.tenants_in_model[m] : 1;
        const int b0 = a.private_mode ? a.bin_base[m] + e * tim : 0;
        int ntile = 0, nshort = 0;
        for (int ul = 0; ul < tim; ++ul) {
            const int cnt = a.private_mode ? a.bin_off[b0 + ul + 1] - a.bin_off[b0 + ul] : expert_off[i + 1] - expert_off[i];
            ntile += (cnt + a.tile_rows - 1) / a.tile_rows;
            const int rem = cnt % a.tile_rows;          // only the last tile of a segment is ragged
            if (rem > 0 && rem <= a.short_rows) ++nshort;
        }
        s_tile_base[i] = ntile;
        s_short_base[i] = nshort;
    }
    __syncthreads();
    const int n_tiles = block_scan_exclusive(s_tile_base, ME, s_warp);
    const int n_short_tiles = simple ? 0 : block_scan_exclusive(s_short_base, ME, s_warp);
    const int n_long_tiles = n_tiles - n_short_tiles;
    if (!general) {
        for (int gidx = tid; gidx <= NG; gidx += nth) {
            int vt = n_tiles, vs = n_short_tiles;
            if (gidx < NG) {
                const int m = gidx / B, b = gidx - m * B;
                vt = s_tile_base[m * a.E + b * a.G];
                vs = simple ? 0 : s_short_base[m * a.E + b * a.G];
            }
            s_group_long0[gidx] = vt - vs;
            s_group_short0[gidx] = vs;
        }
    }
    // per block: its long and its short tiles, then the first tile of every block inside each class
    for (int gidx = tid; gidx < NG && general; gidx += nth) {
        const int m = gidx / B;
        int nt = 0, ns = 0;
        for (int e = 0; e < a.E; ++e) {
            if (block_of(m, e) != gidx) continue;
            const int i = m * a.E + e;
            nt += (i + 1 < ME ? s_tile_base[i + 1] : n_tiles) - s_tile_base[i];
            ns += (i + 1 < ME ? s_short_base[i + 1] : n_short_tiles) - s_short_base[i];
        }
        s_group_long0[gidx] = nt - ns;
        s_group_short0[gidx] = ns;
    }
    if (tid == 0 && general) { s_group_long0[NG] = 0; s_group_short0[NG] = 0; }
    if (general) {
        __syncthreads();
        block_scan_exclusive(s_group_long0, NG + 1, s_warp);
        block_scan_exclusive(s_group_short0, NG + 1, s_warp);
    }
    for (int i = tid; i < ME; i += nth) {
        const int m = i / a.E, e = i - m * a.E;
        const int tim = a.private_mode ? a.tenants_in_model[m] : 1;
        const int b0 = a.private_mode ? a.bin_base[m] + e * tim : 0;
        const int g = block_of(m, e);
        // tiles of the same block and class that belong to earlier experts
        int lix = 0, six = 0;
        for (int e2 = 0; e2 < e && general; ++e2) {
            if (block_of(m, e2) != g) continue;
            const int j = m * a.E + e2;
            const int nt = s_tile_base[j + 1] - s_tile_base[j], ns = s_short_base[j + 1] - s_short_base[j];
            lix += nt - ns;
            six += ns;
        }
        int tix = s_tile_base[i];
        for (int ul = 0; ul < tim; ++ul) {
            const int row_begin = a.private_mode ? a.bin_off[b0 + ul] : expert_off[i];
            const int row_end = a.private_mode ? a.bin_off[b0 + ul + 1] : expert_off[i + 1];
            for (int r = row_begin; r < row_end; r += a.tile_rows, ++tix) {
                Tile t;
                t.row0 = r;
                t.nrows = min(a.tile_rows, row_end - r);
                t.slot = a.slot_table[i];
                t.group = g;
                a.tiles[tix] = t;
                if (general) a.tile_cidx[tix] = (t.nrows <= a.short_rows) ? six++ : lix++;   // rank inside (block, class)
            }
        }
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
        // routed units: the long tiles first, then the short ones; inside each class ordered by (expert block,
        // weight-row block, tile), so that all experts of a block advance through the same weight-row block together
        const int nmax = n_tiles * max(a.nblk1, a.nblk2);
        for (int i = tid; i < nmax; i += nth) {
            const int tile = i % n_tiles, cb = i / n_tiles;
            int c0, nc, ci, base = 0;
            if (simple) {
                // expert block of the tile: last block whose first tile is <= tile (empty blocks share their first
                // tile with the next one)
                int lo = 0, hi = NG;
                while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_group_long0[mid] <= tile) lo = mid; else hi = mid; }
                c0 = s_group_long0[lo]; nc = s_group_long0[lo + 1] - c0; ci = tile - c0;
            } else if (ranged) {
                // the expert of the tile: last expert whose first tile is <= tile (experts without tiles share theirs
                // with the next one)
                int lo = 0, hi = ME;
                while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_tile_base[mid] <= tile) lo = mid; else hi = mid; }
                const int m = lo / a.E, e = lo - m * a.E, g = m * B + e / a.G;
                const int t_end = lo + 1 < ME ? s_tile_base[lo + 1] : n_tiles;
                const int has_short = (lo + 1 < ME ? s_short_base[lo + 1] : n_short_tiles) - s_short_base[lo];
                const bool is_short = has_short && tile == t_end - 1;                 // only an expert's last tile can be short
                const int32_t* g0 = is_short ? s_group_short0 : s_group_long0;
                c0 = g0[g]; nc = g0[g + 1] - c0;
                ci = (is_short ? s_short_base[lo] : tile - s_short_base[lo]) - c0;    // index inside the class, then inside the block
                base = is_short ? n_long_tiles : 0;
            } else {
                const Tile t = a.tiles[tile];
                const bool is_short = t.nrows <= a.short_rows;
                ci = a.tile_cidx[tile];                                 // rank of the tile inside (block, class)
                const int32_t* g0 = is_short ? s_group_short0 : s_group_long0;
                c0 = g0[t.group]; nc = g0[t.group + 1] - c0;            // tiles of earlier blocks in this class, tiles of this block
                base = is_short ? n_long_tiles : 0;
            }
            Unit u; u.colblock = cb * (tm ? 4 : 1); u.tile = tile;
            if (cb < a.nblk1) a.units1[su1 + (base + c0) * a.nblk1 + cb * nc + ci] = u;
            if (cb < a.nblk2) a.units2[su2 + (base + c0) * a.nblk2 + cb * nc + ci] = u;
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
            a.plan_counts[8] = n_short_tiles * a.nblk1;     // units at the tail of the lists that the background lanes may take
            a.plan_counts[9] = n_short_tiles * a.nblk2;
        }
        if (a.token_major) {
            // U equally long units on S CTAs take ceil(U / S) rounds.  The units of the last, partly filled round (the
            // tail of the list: routed ones) are split into units of half the weight rows each (tiles of at most 64
            // rows; narrower units pack more K slices into a stage and stream as fast per byte) whenever the pieces
            // fill fewer (shorter) rounds than the round they replace: 627 units on 148 CTAs = 4 full rounds + 35
            // units; as 70 halves these cost half a round.
            __shared__ int s_split[4];
            int r2[2], f2[2];
            for (int l = 0; l < 2; ++l) {
                const int routed = n_tiles * (l ? a.nblk2 : a.nblk1);
                const int total = (l ? su2 : su1) + routed;
                int r = total % a.n_ctas;
                // pieces per unit when every tile is as small as the batch (direct mode); otherwise halves at most
                // (quarters -- possible where every tile has at most 32 rows and K / 64 is divisible by 4 -- were measured
                // slower than halves at the 32-token decode layer, 110.4 against 107.6 us for gate/up: their eight stages
                // per unit do not cover the fill of the pipeline; the code below would take them with f = 4)
                const int f = 2;
                const int rounds_f = (f * r + a.n_ctas - 1) / a.n_ctas;          // rounds of 1/f length the pieces take
                if (rounds_f >= f || r > routed || r > 128 || !a.split_ok[l]) r = 0;
                r2[l] = r; f2[l] = f;
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
                    cnt = (f2[l] == 4 && rows <= 32) ? 4 : (rows <= 64 ? 2 : 1);
                }
                // position of each unit after the split: the running sum of the extra pieces before it (r <= 128: the
                // first four warps hold them all)
                const int extra = cnt > 0 ? cnt - 1 : 0;
                int incl = extra;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if ((tid & 31) >= o) incl += v;
                }
                if (tid < 128 && (tid & 31) == 31) s_split[tid >> 5] = incl;
                __syncthreads();
                if (tid < r) {
                    int off = tid + incl - extra;
                    for (int w = 0; w < (tid >> 5); ++w) off += s_split[w];
                    // pieces of 256 / cnt weight rows: colblocks count steps of 64 rows, the width code sits in the top byte
                    const int step = 4 / cnt, code = cnt == 4 ? 2 : (cnt == 2 ? 1 : 0);
                    for (int q = 0; q < cnt; ++q) {
                        Unit u = mine;
                        u.colblock = (mine.colblock + q * step) | (code << 24);
                        list[total - r + off + q] = u;
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
        a.plan_counts[4] = 0; a.plan_counts[5] = 0;           // work counters of the two grouped GEMM launches:
        a.plan_counts[10] = 0; a.plan_counts[11] = 0; a.plan_counts[12] = 0; a.plan_counts[13] = 0;         //   two words each (units taken from the front of the
                                                              //   list, units taken from its tail)
    }
}

}  // namespace faasmoe
