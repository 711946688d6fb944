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
    a.tile_rows = pair ? (tc_wide_mode(c, T) ? 512 : 256) : kTileRows;
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
    a.direct = tc_direct_mode(c, T) ? 1 : 0;
    a.interleave_down = (a.token_major && g.shared_inter > 0 &&
                         (long long)a.shared_down_width * g.shared_inter == 256ll * g.inter) ? 1 : 0;
    a.tiles = c->ws.tiles; a.stiles = c->ws.stiles;
    a.units1 = tc ? c->ws.units1 : nullptr; a.units2 = tc ? c->ws.units2 : nullptr;
    a.plan_counts = c->ws.plan_counts;
    return a;
}

size_t plan_smem_ints(const moe_ctx* c, int G)
{
    const moe_config& g = c->cfg;
    const int B = (g.n_experts + G - 1) / G;
    return (size_t)g.n_models * g.n_experts + (size_t)g.n_models * B + 1;
}

cudaError_t launch_plan(moe_ctx* c, const int32_t* expert_off, int T, int G, bool with_shared, cudaStream_t st)
{
    const PlanArgs a = make_plan_args(c, T, G, with_shared);
    launch_pdl(plan_kernel, dim3(1), dim3(512), plan_smem_ints(c, G) * sizeof(int32_t), st, expert_off, a);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
