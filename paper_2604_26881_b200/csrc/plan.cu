// Work plan of the expert execution: tiles of rows that share an expert, grouped by expert
// block (paper Sec. 3 / Sec. 5: G experts per function is the granularity at which expert work
// is partitioned), and the unit lists of the tensor-core grouped GEMMs.
#include "internal.h"
#include "plan.cuh"

namespace faasmoe {

namespace {

__global__ void __launch_bounds__(512)
plan_kernel(const int32_t* __restrict__ expert_off, PlanArgs a)
{
    extern __shared__ int32_t s_mem[];
    __shared__ int32_t s_warp[33];
    pdl_wait();
    pdl_launch_dependents();
    plan_body(expert_off, a, s_mem, s_warp);
}

// Tiles and unit lists of the shared expert alone, for one model: none of it depends on the routing, so these units
// can run while the router and the dispatch are still at work (same order and encoding as in plan_body).
__global__ void __launch_bounds__(256)
plan_shared_kernel(PlanArgs a)
{
    pdl_wait();
    pdl_launch_dependents();
    const int tid = threadIdx.x, nth = blockDim.x;
    const int n_stiles = (a.T + a.tile_rows - 1) / a.tile_rows;
    for (int i = tid; i < n_stiles; i += nth) {
        Tile t;
        t.row0 = i * a.tile_rows;
        t.nrows = min(a.tile_rows, a.T - t.row0);
        t.slot = 0;
        t.group = 0;
        a.stiles[i] = t;
    }
    const int su1 = n_stiles * a.snblk1, su2 = n_stiles * a.snblk2;
    const int tm = a.token_major;
    const int wsh = a.shared_down_width;
    const int sh_step = wsh / 64, sh_code = wsh == 256 ? 0 : (wsh == 128 ? 1 : 2);
    for (int i = tid; i < su1; i += nth) {
        Unit u;
        u.colblock = (i / n_stiles) * (tm ? 4 : 1);
        u.tile = ~(i % n_stiles);
        a.units1[i] = u;
    }
    for (int i = tid; i < su2; i += nth) {
        Unit u;
        const int cb = i / n_stiles;
        u.colblock = tm ? (cb * sh_step) | (sh_code << 24) : cb;
        u.tile = ~(i % n_stiles);
        a.units2[i] = u;
    }
    if (tid == 0) {
        a.plan_counts[0] = 0; a.plan_counts[1] = n_stiles;
        a.plan_counts[2] = su1; a.plan_counts[3] = su2;
        a.plan_counts[4] = 0; a.plan_counts[5] = 0;     // work counters
        a.plan_counts[6] = 0; a.plan_counts[7] = 0;     // nothing to deal out between routed units
        a.plan_counts[8] = 0; a.plan_counts[9] = 0;     // no short units
        a.plan_counts[10] = 0; a.plan_counts[11] = 0; a.plan_counts[12] = 0; a.plan_counts[13] = 0;
    }
}

}  // namespace

PlanArgs make_plan_args(moe_ctx* c, int T, int G, bool with_shared)
{
    const moe_config& g = c->cfg;
    const bool tc = tc_supported(c);
    // weight-row blocks per unit: gate/up 64 intermediate indices, down 128 rows; a CTA pair takes two
    const bool pair = tc && tc_pair_mode(c, T);
    const bool wide_rows = pair || (tc && tc_token_major(c, T));      // 256 weight rows per unit
    const int div1 = wide_rows ? 128 : 64, div2 = wide_rows ? 256 : 128;
    PlanArgs a;
    a.slot_table = c->d_slot;
    a.M = g.n_models; a.E = g.n_experts; a.G = G; a.T = T;
    a.tile_rows = pair ? (tc_wide_mode(c, T) ? (tc_background_mode(c, T) ? 2 * kAccRowsBg : 512) : 256) : kTileRows;
    a.model_tok_off = g.n_models > 1 ? c->ws.model_tok_off : nullptr;
    a.with_shared = with_shared ? 1 : 0;
    a.nblk1 = g.inter / div1; a.nblk2 = g.hidden / div2;
    a.snblk1 = g.shared_inter / div1; a.snblk2 = g.hidden / div2;
    a.token_major = (tc && tc_token_major(c, T)) ? 1 : 0;
    a.n_ctas = c->sm_count;
    a.shared_down_width = 256;
    if (a.token_major && g.shared_inter > 0) {
        // few tokens: the shared expert's down units get narrower (their K slices per stage must divide K / 64)
        const int want = T <= 32 ? 64 : (T <= 64 ? 128 : 256);
        if ((g.shared_inter / 64) % (256 / want) == 0) a.shared_down_width = want;
        a.snblk2 = g.hidden / a.shared_down_width;
    }
    a.split_ok[0] = (g.hidden / 64) % 2 == 0; a.split_ok[1] = (g.inter / 64) % 2 == 0;
    a.split4_ok[0] = (g.hidden / 64) % 4 == 0; a.split4_ok[1] = (g.inter / 64) % 4 == 0;
    a.direct = tc_direct_mode(c, T) ? 1 : 0;
    a.interleave_down = (a.token_major && g.shared_inter > 0 &&
                         (long long)a.shared_down_width * g.shared_inter == 256ll * g.inter) ? 1 : 0;
    // pair shape: tiles of at most kShortRows rows are kept apart for the background lanes of the grouped GEMM
    a.short_rows = (pair && tc_background_mode(c, T)) ? kShortRows : 0;
    a.tile_cidx = c->ws.tile_cidx;
    a.block_table = c->d_block_table; a.table_blocks = c->table_blocks;
    a.private_mode = c->dispatch_private;
    a.bin_off = c->ws.bin_off; a.bin_base = c->d_bin_base; a.tenants_in_model = c->d_tenants_in_model;
    a.tiles = c->ws.tiles; a.stiles = c->ws.stiles;
    a.units1 = tc ? c->ws.units1 : nullptr; a.units2 = tc ? c->ws.units2 : nullptr;
    a.plan_counts = c->ws.plan_counts;
    return a;
}

size_t plan_smem_ints(const moe_ctx* c, int G)
{
    const moe_config& g = c->cfg;
    const int B = c->d_block_table ? c->table_blocks : (g.n_experts + G - 1) / G;
    return 2 * ((size_t)g.n_models * g.n_experts + (size_t)g.n_models * B + 1);
}

cudaError_t launch_plan(moe_ctx* c, const int32_t* expert_off, int T, int G, bool with_shared, cudaStream_t st)
{
    const PlanArgs a = make_plan_args(c, T, G, with_shared);
    launch_pdl(plan_kernel, dim3(1), dim3(512), plan_smem_ints(c, G) * sizeof(int32_t), st, expert_off, a);
    c->launches += 1;
    return cudaGetLastError();
}

void shared_unit_counts(moe_ctx* c, int T, int* n_units1, int* n_units2)
{
    PlanArgs a = make_plan_args(c, T, 1, true);
    if (tc_background_mode(c, T)) a.tile_rows = 512;
    const int n_stiles = (T + a.tile_rows - 1) / a.tile_rows;
    *n_units1 = n_stiles * a.snblk1;
    *n_units2 = n_stiles * a.snblk2;
}

cudaError_t launch_plan_shared(moe_ctx* c, int T, cudaStream_t st)
{
    PlanArgs a = make_plan_args(c, T, 1, true);
    if (tc_background_mode(c, T)) a.tile_rows = 512;      // launched in the shape without the background pipeline
    a.stiles = c->ws.stiles_sh; a.units1 = c->ws.units1_sh; a.units2 = c->ws.units2_sh;
    a.plan_counts = c->ws.plan_counts_sh;
    launch_pdl(plan_shared_kernel, dim3(1), dim3(256), 0, st, a);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
