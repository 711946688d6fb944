// Work plan of the expert execution: tiles of rows that share an expert, grouped by expert
// block (paper Sec. 3 / Sec. 5: G experts per function is the granularity at which expert work
// is partitioned), and the unit lists of the tensor-core grouped GEMMs.
#include "internal.h"

namespace faasmoe {

namespace {

// Exclusive scan of data[0..n) in shared memory by one block; returns the total.
__device__ int block_exclusive_scan(int32_t* data, int n, int32_t* s_part /* [blockDim.x] */)
{
    const int tid = threadIdx.x, nth = blockDim.x;
    const int per = (n + nth - 1) / nth;
    const int b0 = min(n, tid * per), b1 = min(n, b0 + per);
    int sum = 0;
    for (int b = b0; b < b1; ++b) sum += data[b];
    s_part[tid] = sum;
    __syncthreads();
    for (int off = 1; off < nth; off <<= 1) {
        const int v = (tid >= off) ? s_part[tid - off] : 0;
        __syncthreads();
        s_part[tid] += v;
        __syncthreads();
    }
    int run = s_part[tid] - sum;
    const int total = s_part[nth - 1];
    for (int b = b0; b < b1; ++b) { const int c = data[b]; data[b] = run; run += c; }
    __syncthreads();
    return total;
}

// One block.  ME = M*E experts; groups are blocks of G consecutive experts of one model.
__global__ void __launch_bounds__(512)
plan_kernel(const int32_t* __restrict__ expert_off, const int32_t* __restrict__ slot_table, int M, int E, int G, int T,
            int tile_rows, const int32_t* __restrict__ model_tok_off /* null when M == 1 */, bool with_shared,
            int nblk1 /* weight-row blocks of the gate/up GEMM, routed */, int nblk2 /* down GEMM */,
            int snblk1, int snblk2, Tile* __restrict__ tiles, Tile* __restrict__ stiles, Unit* __restrict__ units1,
            Unit* __restrict__ units2, int32_t* __restrict__ plan_counts)
{
    extern __shared__ int32_t s_mem[];
    const int ME = M * E;
    const int B = (E + G - 1) / G;
    const int NG = M * B;
    int32_t* s_tile_base = s_mem;            // [ME]   tiles before expert i
    int32_t* s_group_tile0 = s_mem + ME;     // [NG+1] first tile of each group
    __shared__ int32_t s_part[512];
    const int tid = threadIdx.x, nth = blockDim.x;

    for (int i = tid; i < ME; i += nth) {
        const int cnt = expert_off[i + 1] - expert_off[i];
        s_tile_base[i] = (cnt + tile_rows - 1) / tile_rows;
    }
    __syncthreads();
    const int n_tiles = block_exclusive_scan(s_tile_base, ME, s_part);
    for (int i = tid; i < ME; i += nth) {
        const int m = i / E, e = i - m * E;
        const int row_begin = expert_off[i], row_end = expert_off[i + 1];
        int tix = s_tile_base[i];
        for (int r = row_begin; r < row_end; r += tile_rows, ++tix) {
            Tile t;
            t.row0 = r;
            t.nrows = min(tile_rows, row_end - r);
            t.slot = slot_table[i];
            t.group = m * B + e / G;
            tiles[tix] = t;
        }
    }
    for (int gidx = tid; gidx <= NG; gidx += nth) {
        int v = n_tiles;
        if (gidx < NG) {
            const int m = gidx / B, b = gidx - m * B;
            v = s_tile_base[m * E + b * G];
        }
        s_group_tile0[gidx] = v;
    }
    __syncthreads();

    // shared-expert tiles: tokens of one model, kTileRows at a time
    int n_stiles = 0;
    if (with_shared) {
        for (int m = 0; m < M; ++m) {
            const int t_begin = model_tok_off ? model_tok_off[m] : 0;
            const int t_end = model_tok_off ? model_tok_off[m + 1] : T;
            const int nt = (t_end - t_begin + tile_rows - 1) / tile_rows;
            for (int i = tid; i < nt; i += nth) {
                Tile t;
                t.row0 = t_begin + i * tile_rows;
                t.nrows = min(tile_rows, t_end - t.row0);
                t.slot = m;
                t.group = m;
                stiles[n_stiles + i] = t;
            }
            n_stiles += nt;
        }
    }

    // Unit lists of the grouped GEMMs.  Shared-expert units come first (uniform, large), then
    // the routed units ordered by (expert block, weight-row block, tile): all experts of a
    // block advance through the same weight-row block together.
    if (units1) {
        const int su1 = n_stiles * snblk1, su2 = n_stiles * snblk2;
        for (int i = tid; i < su1; i += nth) { Unit u; u.colblock = i / n_stiles; u.tile = ~(i % n_stiles); units1[i] = u; }
        for (int i = tid; i < su2; i += nth) { Unit u; u.colblock = i / n_stiles; u.tile = ~(i % n_stiles); units2[i] = u; }
        __syncthreads();                      // the tiles written above are read back below
        for (int i = tid; i < n_tiles * nblk1; i += nth) {
            const int tile = i % n_tiles, cb = i / n_tiles;
            const int gidx = tiles[tile].group;
            const int t0 = s_group_tile0[gidx], nt = s_group_tile0[gidx + 1] - t0;
            Unit u; u.colblock = cb; u.tile = tile;
            units1[su1 + t0 * nblk1 + cb * nt + (tile - t0)] = u;
        }
        for (int i = tid; i < n_tiles * nblk2; i += nth) {
            const int tile = i % n_tiles, cb = i / n_tiles;
            const int gidx = tiles[tile].group;
            const int t0 = s_group_tile0[gidx], nt = s_group_tile0[gidx + 1] - t0;
            Unit u; u.colblock = cb; u.tile = tile;
            units2[su2 + t0 * nblk2 + cb * nt + (tile - t0)] = u;
        }
        if (tid == 0) {
            plan_counts[2] = su1 + n_tiles * nblk1;
            plan_counts[3] = su2 + n_tiles * nblk2;
        }
    }
    if (tid == 0) {
        plan_counts[0] = n_tiles;
        plan_counts[1] = n_stiles;
        plan_counts[4] = 0;           // work counters of the two grouped GEMM launches
        plan_counts[5] = 0;
    }
}

}  // namespace

cudaError_t launch_plan(moe_ctx* c, const int32_t* expert_off, int T, int G, bool with_shared, cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const int ME = g.n_models * g.n_experts;
    const int B = (g.n_experts + G - 1) / G;
    const size_t smem = (size_t)(ME + g.n_models * B + 1) * sizeof(int32_t);
    const bool tc = tc_supported(c);
    // weight-row blocks per unit: gate/up 64 intermediate indices, down 128 rows; a CTA pair takes two
    const bool pair = tc && tc_pair_mode(c, T);
    const int div1 = pair ? 128 : 64, div2 = pair ? 256 : 128;
    const int nblk1 = g.inter / div1, nblk2 = g.hidden / div2;
    const int snblk1 = g.shared_inter / div1, snblk2 = g.hidden / div2;
    const int tile_rows = pair ? 256 : kTileRows;
    plan_kernel<<<1, 512, smem, st>>>(expert_off, c->d_slot, g.n_models, g.n_experts, G, T, tile_rows,
                                      g.n_models > 1 ? c->ws.model_tok_off : nullptr, with_shared, nblk1, nblk2,
                                      snblk1, snblk2, c->ws.tiles, c->ws.stiles, tc ? c->ws.units1 : nullptr,
                                      tc ? c->ws.units2 : nullptr, c->ws.plan_counts);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
