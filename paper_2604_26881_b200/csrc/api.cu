// C-ABI entry points: argument validation, context and workspace management, call sequencing.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"
#include "plan.cuh"

using namespace faasmoe;

namespace {

thread_local char g_last_cuda_error[256] = "";


#define MOE_CUDA(ctx, expr)                                                                         \
    do {                                                                                            \
        cudaError_t err__ = (expr);                                                                 \
        if (err__ != cudaSuccess) {                                                                 \
            snprintf((ctx)->errbuf, sizeof((ctx)->errbuf), "%.160s: %s", #expr, cudaGetErrorString(err__)); \
            snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s", (ctx)->errbuf);           \
            return MOE_ERR_CUDA;                                                                    \
        }                                                                                           \
    } while (0)

template <typename T>
cudaError_t dev_alloc(T** p, size_t n)
{
    *p = nullptr;
    if (n == 0) n = 1;
    return cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T));
}

int div_up(int a, int b) { return (a + b - 1) / b; }

// Activation and output buffers are read and written with 16-byte vector accesses (and as TMA tiles), so a pointer
// that is not 16-byte aligned is refused on the host: a kernel given one would fault.
template <typename... P>
bool misaligned16(P... ptrs)
{
    uintptr_t bits = 0;
    ((bits |= (uintptr_t)ptrs), ...);
    return (bits & 15u) != 0;
}

int alloc_workspace(moe_ctx* c)
{
    const moe_config& g = c->cfg;
    Workspace& w = c->ws;
    const size_t T = g.max_tokens, k = g.top_k, R = T * k, H = g.hidden, I = g.inter, Is = g.shared_inter;
    const size_t ME = (size_t)g.n_models * g.n_experts;
    c->nbins = g.n_experts * g.n_tenants;
    c->nblk_rows = div_up((int)R, kDispatchChunk);
    c->nblk_tok = div_up((int)T, kDispatchChunk);
    // (+ one ragged tile per expert; per (tenant, expert) bin when private orchestrators keep the tenants' rows apart)
    c->max_tiles = div_up((int)R, kTileRows) + std::max((int)ME, c->nbins);
    c->max_stiles = div_up((int)T, kTileRows) + g.n_models;
    const int nblk1 = g.inter / 64, nblk2 = div_up(g.hidden, 128), snblk1 = g.shared_inter / 64;
    // (+512: the token-major plan splits up to 128 units of the last round in two or four; its shared units are up to
    // 4x narrower)
    c->max_units1 = c->max_tiles * nblk1 + c->max_stiles * snblk1 + 512;
    c->max_units2 = (c->max_tiles + 4 * c->max_stiles) * nblk2 + 512;

    cudaError_t e = cudaSuccess;
    auto A = [&](auto** p, size_t n) { if (e == cudaSuccess) e = dev_alloc(p, n); };
    A(&w.topk_idx, R); A(&w.topk_w, R); A(&w.shared_gate, T); A(&w.tie_flag, T);
    A(&w.perm, R); A(&w.inv_perm, R); A(&w.tenant_expert_count, (size_t)g.n_tenants * g.n_experts);
    A(&w.expert_off, ME + 1); A(&w.group_off, ME + 1);
    A(&w.block_cnt, (size_t)c->nblk_rows * c->nbins); A(&w.bin_off, (size_t)c->nbins + 1);
    A(&w.tok_block_cnt, (size_t)c->nblk_tok * g.n_models); A(&w.model_tok_off, (size_t)g.n_models + 1);
    A(&w.tok_perm, T); A(&w.tok_inv, T);
    A(&w.tiles, (size_t)c->max_tiles); A(&w.tile_cidx, (size_t)c->max_tiles); A(&w.stiles, (size_t)c->max_stiles); A(&w.plan_counts, 16);
    A(&w.units1, (size_t)c->max_units1); A(&w.units2, (size_t)c->max_units2);
    if (Is > 0 && g.n_models == 1) {
        A(&w.stiles_sh, (size_t)c->max_stiles); A(&w.plan_counts_sh, 16);
        A(&w.units1_sh, (size_t)c->max_stiles * snblk1); A(&w.units2_sh, (size_t)4 * c->max_stiles * nblk2);
    }
    // activations: one extra tile of rows so that a whole-tile load never leaves the buffer
    A(&w.x_perm, (R + kTileRows) * H); A(&w.h, (R + kTileRows) * I); A(&w.y_perm, R * H);
    if (g.n_models > 1) A(&w.xs_perm, (T + kTileRows) * H);
    if (Is > 0) {
        bf16* hs16 = nullptr;                       // same element size as fp16
        A(&hs16, (T + kTileRows) * Is);
        w.hs = hs16;
        A(&w.y_shared, T * H);
    }
    A(&w.xn, (T + kTileRows) * H);
    A(&w.x_stage, (T + kTileRows) * H); A(&w.tenant_stage, T); A(&w.out_stage, T * H);
    A(&w.x_stage2, (T + kTileRows) * H); A(&w.tenant_stage2, T); A(&w.out_stage2, T * H);
    A(&w.status, 1); A(&w.stats, 4); A(&w.dispatch_done, 1);
    if (e != cudaSuccess) {
        snprintf(c->errbuf, sizeof(c->errbuf), "workspace allocation: %s", cudaGetErrorString(e));
        return MOE_ERR_ALLOC;
    }
    cudaMemset(w.status, 0, sizeof(int32_t));
    cudaMemset(w.stats, 0, 4 * sizeof(int32_t));
    cudaMemset(w.dispatch_done, 0, sizeof(int32_t));
    cudaMemset(w.plan_counts, 0, 16 * sizeof(int32_t));
    if (w.plan_counts_sh) cudaMemset(w.plan_counts_sh, 0, 16 * sizeof(int32_t));
    return MOE_OK;
}

void free_workspace(moe_ctx* c)
{
    Workspace& w = c->ws;
    void* ptrs[] = {w.topk_idx, w.topk_w, w.shared_gate, w.tie_flag, w.perm, w.inv_perm, w.tenant_expert_count,
                    w.expert_off, w.group_off, w.block_cnt, w.bin_off, w.tok_block_cnt, w.model_tok_off, w.tok_perm,
                    w.tok_inv, w.tiles, w.tile_cidx, w.stiles, w.plan_counts, w.units1, w.units2, w.stiles_sh, w.plan_counts_sh, w.units1_sh,
                    w.units2_sh, w.x_perm, w.xs_perm, w.h, w.hs,
                    w.y_perm, w.y_shared, w.xn, w.x_stage, w.tenant_stage, w.out_stage, w.x_stage2, w.tenant_stage2, w.out_stage2,
                    w.status, w.stats, w.dispatch_done};
    for (void* p : ptrs) if (p) cudaFree(p);
    w = Workspace();
}

// Uploads the tenant -> model table and the bin layout derived from it.
int upload_tenant_tables(moe_ctx* c)
{
    const moe_config& g = c->cfg;
    std::vector<int32_t> local(g.n_tenants), per_model(g.n_models, 0), base(g.n_models + 1, 0);
    for (int u = 0; u < g.n_tenants; ++u) local[u] = per_model[c->h_model_of_tenant[u]]++;
    for (int m = 0; m < g.n_models; ++m) base[m + 1] = base[m] + g.n_experts * per_model[m];
    MOE_CUDA(c, cudaMemcpy(c->d_model_of_tenant, c->h_model_of_tenant.data(), sizeof(int32_t) * g.n_tenants,
                           cudaMemcpyHostToDevice));
    MOE_CUDA(c, cudaMemcpy(c->d_tenant_local, local.data(), sizeof(int32_t) * g.n_tenants, cudaMemcpyHostToDevice));
    MOE_CUDA(c, cudaMemcpy(c->d_tenants_in_model, per_model.data(), sizeof(int32_t) * g.n_models,
                           cudaMemcpyHostToDevice));
    MOE_CUDA(c, cudaMemcpy(c->d_bin_base, base.data(), sizeof(int32_t) * (g.n_models + 1), cudaMemcpyHostToDevice));
    return MOE_OK;
}

// The tensor-core gate/up kernel reads W_gate and W_up through ONE 3-D TMA map whose middle dimension steps from one
// array to the other, so the distance between the two arrays becomes a stride of the map: it must be a non-zero
// multiple of 16 bytes below 2^40.
bool pair_distance_ok(const void* a, const void* b)
{
    const uintptr_t pa = (uintptr_t)a, pb = (uintptr_t)b;
    const uintptr_t diff = pa < pb ? pb - pa : pa - pb;
    return diff != 0 && (diff & 15) == 0 && diff < (1ull << 40);
}

int check_layer_ready(const moe_ctx* c, int layer, bool need_pool, bool need_shared)
{
    if (layer < 0 || layer >= c->cfg.n_layers) return MOE_ERR_SHAPE;
    if (need_pool && !c->pool_set[layer]) return MOE_ERR_STATE;
    for (int m = 0; m < c->cfg.n_models; ++m) {
        if (!c->model_set[(size_t)layer * c->cfg.n_models + m]) return MOE_ERR_STATE;
        if (need_shared && c->cfg.shared_inter > 0 && !c->models[(size_t)layer * c->cfg.n_models + m].ws_gate)
            return MOE_ERR_STATE;
    }
    return MOE_OK;
}

bool use_tc(const moe_ctx* c)
{
    if (c->expert_path == MOE_PATH_FMA) return false;
    return tc_supported(c);
}

int experts_impl(moe_ctx* c, int layer, const bf16* x, const bf16* x_perm, const int32_t* perm,
                 const int32_t* expert_off, const int32_t* tenant_id, int T, int G, float* y_perm, float* y_shared,
                 cudaStream_t st, bool plan_done = false, bool sort_done = false, bool tokens_ready = false)
{
    const moe_config& g = c->cfg;
    const bool with_shared = y_shared != nullptr && g.shared_inter > 0;
    const bf16* xs = x;
    const int32_t* dst_rows = nullptr;
    if (with_shared && g.n_models > 1) {
        if (!sort_done) MOE_CUDA(c, launch_token_sort(c, x, tenant_id, T, st));
        xs = c->ws.xs_perm;
        dst_rows = c->ws.tok_perm;
    }
    if (!plan_done) MOE_CUDA(c, launch_plan(c, expert_off, T, G, with_shared, st));
    stage_mark(c, st, kEvPlan);
    if (use_tc(c)) {
        const int rc = tc_setup_layer(c, layer);
        if (rc != MOE_OK) return rc;
        MOE_CUDA(c, launch_experts_tc(c, layer, xs, x_perm, perm, T, y_perm, with_shared ? y_shared : nullptr, dst_rows,
                                      st, false, tokens_ready));
    } else {
        MOE_CUDA(c, launch_experts_fma(c, layer, xs, x_perm, T, y_perm, with_shared ? y_shared : nullptr, dst_rows, st));
    }
    return MOE_OK;
}

int layer_forward_impl(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int G,
                       const bf16* residual, bf16* out, cudaStream_t st, bool routed = false)
{
    const moe_config& g = c->cfg;
    Workspace& w = c->ws;
    const bool shared = g.shared_inter > 0;
    // One model: the shared expert's work does not depend on the routing.  Its two launches go to a second stream, where
    // they run beside the router and the dispatch (HBM- or tensor-bound work beside latency-bound work); the combine
    // waits for both streams.  By default only for batches of the 2-CTA shape: with fewer tokens the two event
    // edges cost what the overlap gains.  Not while the stages are being timed one by one.
    const bool early = shared && g.n_models == 1 && use_tc(c) && !c->timing && c->side != nullptr &&
                       (c->early_shared_enabled == 2 || (c->early_shared_enabled == 1 && tc_pair_mode(c, T)));
    if (early) {
        const int rc = tc_setup_layer(c, layer);
        if (rc != MOE_OK) return rc;
        MOE_CUDA(c, cudaEventRecord(c->ev_fork, st));
        MOE_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        MOE_CUDA(c, launch_plan_shared(c, T, c->side));
        MOE_CUDA(c, launch_experts_tc(c, layer, x, nullptr, nullptr, T, nullptr, w.y_shared, nullptr, c->side, true));
        MOE_CUDA(c, cudaEventRecord(c->ev_join, c->side));
    }
    // Several models: the shared experts read the tokens grouped by model.  That grouping (four small launches) depends
    // on the tenant ids only and runs on the second stream beside the router and the dispatch; the plan waits for it.
    const bool sort_early = shared && g.n_models > 1 && !c->timing && c->side != nullptr && c->early_shared_enabled != 0;
    if (sort_early) {
        MOE_CUDA(c, cudaEventRecord(c->ev_fork, st));
        MOE_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        MOE_CUDA(c, launch_token_sort(c, x, tenant_id, T, c->side));
        MOE_CUDA(c, cudaEventRecord(c->ev_join, c->side));
    }
    stage_mark(c, st, kEvBegin);
    // with few tokens the tensor-core experts read the tokens in place: no permuted copy to make
    const bool direct = use_tc(c) && tc_direct_mode(c, T);
    bool plan_done = false, dispatched = false;
    // (routed: the gate has run already and its results are in the workspace -- the paged entry point looks at them first)
    if (!routed)
        MOE_CUDA(c, launch_route_dispatch(c, layer, x, tenant_id, T, G, w.topk_idx, w.topk_w, shared ? w.shared_gate : nullptr,
                                          w.tie_flag, w.perm, w.inv_perm, w.tenant_expert_count, w.expert_off, w.group_off,
                                          direct ? nullptr : w.x_perm, st, shared && !early, &dispatched, &plan_done));
    stage_mark(c, st, kEvRoute);
    // (a batch that one CTA routes has been dispatched by that CTA)
    if (!dispatched)
        MOE_CUDA(c, launch_dispatch(c, x, w.topk_idx, tenant_id, T, G, w.perm, w.inv_perm, w.tenant_expert_count,
                                    w.expert_off, w.group_off, direct ? nullptr : w.x_perm, st, true, shared && !early, &plan_done));
    stage_mark(c, st, kEvDispatch);
    if (sort_early) MOE_CUDA(c, cudaStreamWaitEvent(st, c->ev_join, 0));
    const int rc = experts_impl(c, layer, x, w.x_perm, w.perm, w.expert_off, tenant_id, T, G, w.y_perm,
                                (shared && !early) ? w.y_shared : nullptr, st, plan_done, sort_early,
                                /* the kernels of this pass that run before the experts only read the tokens */ true);
    if (rc != MOE_OK) return rc;
    if (early) MOE_CUDA(c, cudaStreamWaitEvent(st, c->ev_join, 0));
    MOE_CUDA(c, launch_combine(c, w.y_perm, w.inv_perm, w.topk_w, shared ? w.y_shared : nullptr,
                               shared ? w.shared_gate : nullptr, residual, T, out, st));
    stage_mark(c, st, kEvCombine);
    return MOE_OK;
}

// flags the experts that the routed rows of a batch go to
__global__ void mark_active_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ tenant_id,
                                   const int32_t* __restrict__ model_of_tenant, int R, int k, int E, int n_tenants,
                                   int32_t* __restrict__ active)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    const int u = tenant_id[r / k], e = topk_idx[r];
    if (u < 0 || u >= n_tenants || e < 0 || e >= E) return;
    active[model_of_tenant[u] * E + e] = 1;
}

}  // namespace

extern "C" {

int moe_create(const moe_config* cfg, moe_ctx** out)
{
    if (!cfg || !out) return MOE_ERR_NULL;
    *out = nullptr;
    const moe_config& g = *cfg;
    if (g.hidden < 128 || g.hidden % 128 || g.hidden > 8192) return MOE_ERR_SHAPE;
    if (g.inter < 128 || g.inter % 128) return MOE_ERR_SHAPE;
    if (g.shared_inter < 0 || g.shared_inter % 128) return MOE_ERR_SHAPE;
    if (g.n_experts < 1 || g.n_experts > kMaxExperts) return MOE_ERR_SHAPE;
    if (g.top_k < 1 || g.top_k > kMaxTopK || g.top_k > g.n_experts) return MOE_ERR_SHAPE;
    if (g.n_models < 1 || g.n_models > kMaxExperts || g.n_tenants < 1 || g.n_layers < 1 || g.n_slots < 1)
        return MOE_ERR_SHAPE;
    if ((long long)g.n_experts * g.n_tenants > kMaxBins) return MOE_ERR_UNSUPPORTED;
    if (g.max_tokens < 1 || (long long)g.max_tokens * g.top_k > (1 << 28)) return MOE_ERR_SHAPE;
    if (!(g.rms_eps >= 0.f)) return MOE_ERR_SHAPE;

    moe_ctx* c = new (std::nothrow) moe_ctx();
    if (!c) return MOE_ERR_ALLOC;
    c->cfg = g;
    c->expert_path = MOE_PATH_AUTO;
    c->launches = 0;
    c->tmaps = nullptr;
    c->rmaps = nullptr;
    c->route_path = MOE_PATH_AUTO;
    c->route_lanes2 = 1;
    c->pair_mode_enabled = 1;
    c->wide_tiles_enabled = 1;
    c->token_major_enabled = 1;
    c->dispatch_private = 0;
    c->background_enabled = 1;
    c->fused_dispatch_enabled = 0;      // (measured: 1 % slower at 32 tokens, see the header)
    c->head_units_enabled = 1;
    c->timing = false;
    c->early_shared_enabled = 1;
    c->early_shared_sms = 1 << 20;      // no limit
    c->side = nullptr; c->ev_fork = nullptr; c->ev_join = nullptr;
    c->copy_in = nullptr; c->copy_out = nullptr; c->submitted = 0; c->waited[0] = c->waited[1] = -1;
    for (int i = 0; i < 2; ++i) { c->ev_in[i] = nullptr; c->ev_done[i] = nullptr; c->ev_out[i] = nullptr; }
    for (auto& e : c->ev) e = nullptr;
    c->errbuf[0] = 0;
    c->d_models = nullptr; c->d_slot = nullptr; c->d_model_of_tenant = nullptr; c->d_tenant_local = nullptr;
    c->d_bin_base = nullptr; c->d_tenants_in_model = nullptr;
    c->d_block_table = nullptr; c->table_blocks = 0;
    int rc = MOE_OK;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    const size_t LM = (size_t)g.n_layers * g.n_models, ME = (size_t)g.n_models * g.n_experts;
    c->pools.assign(g.n_layers, PoolWeights{nullptr, nullptr, nullptr});
    c->pool_set.assign(g.n_layers, 0);
    c->models.assign(LM, ModelWeights{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr});
    c->model_set.assign(LM, 0);
    c->h_slot.resize(ME);
    for (size_t i = 0; i < ME; ++i) c->h_slot[i] = (int32_t)(i % (size_t)g.n_slots);
    c->h_model_of_tenant.resize(g.n_tenants);
    for (int u = 0; u < g.n_tenants; ++u) c->h_model_of_tenant[u] = u % g.n_models;
    if (e == cudaSuccess) e = dev_alloc(&c->d_models, LM);
    if (e == cudaSuccess) e = dev_alloc(&c->d_slot, ME);
    if (e == cudaSuccess) e = dev_alloc(&c->d_model_of_tenant, (size_t)g.n_tenants);
    if (e == cudaSuccess) e = dev_alloc(&c->d_tenant_local, (size_t)g.n_tenants);
    if (e == cudaSuccess) e = dev_alloc(&c->d_bin_base, (size_t)g.n_models + 1);
    if (e == cudaSuccess) e = dev_alloc(&c->d_tenants_in_model, (size_t)g.n_models);
    if (e == cudaSuccess) e = cudaMemset(c->d_models, 0, LM * sizeof(ModelWeights));
    if (e == cudaSuccess) e = cudaMemcpy(c->d_slot, c->h_slot.data(), ME * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "moe_create: %s", cudaGetErrorString(e));
        rc = MOE_ERR_CUDA;
    }
    if (rc == MOE_OK) rc = upload_tenant_tables(c);
    if (rc == MOE_OK) rc = alloc_workspace(c);
    if (rc == MOE_OK && g.shared_inter > 0) {
        e = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "moe_create: %s", cudaGetErrorString(e));
            rc = MOE_ERR_CUDA;
        }
    }
    if (rc == MOE_OK) {
        e = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking);
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) {
            snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "moe_create: %s", cudaGetErrorString(e));
            rc = MOE_ERR_CUDA;
        }
    }
    if (rc != MOE_OK) {
        if (c->errbuf[0]) snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s", c->errbuf);
        moe_destroy(c);
        return rc;
    }
    *out = c;
    return MOE_OK;
}

int moe_destroy(moe_ctx* c)
{
    if (!c) return MOE_ERR_NULL;
    cudaDeviceSynchronize();
    tc_destroy(c);
    route_tc_destroy(c);
    free_workspace(c);
    for (auto& e : c->ev) if (e) cudaEventDestroy(e);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->side) cudaStreamDestroy(c->side);
    for (int i = 0; i < 2; ++i) {
        if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
        if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
        if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
    }
    if (c->copy_in) cudaStreamDestroy(c->copy_in);
    if (c->copy_out) cudaStreamDestroy(c->copy_out);
    void* ptrs[] = {c->d_models, c->d_slot, c->d_model_of_tenant, c->d_tenant_local, c->d_bin_base,
                    c->d_tenants_in_model, c->d_block_table};
    for (void* p : ptrs) if (p) cudaFree(p);
    if (c->res.d_active) cudaFree(c->res.d_active);
    if (c->res.h_active) cudaFreeHost(c->res.h_active);
    delete c;
    return MOE_OK;
}

int moe_set_expert_pool(moe_ctx* c, int layer, const void* w_gate, const void* w_up, const void* w_down)
{
    if (!c || !w_gate || !w_up || !w_down) return MOE_ERR_NULL;
    if (layer < 0 || layer >= c->cfg.n_layers) return MOE_ERR_SHAPE;
    if (((uintptr_t)w_gate | (uintptr_t)w_up | (uintptr_t)w_down) & 15) return MOE_ERR_SHAPE;
    if (tc_supported(c) && !pair_distance_ok(w_gate, w_up)) return MOE_ERR_UNSUPPORTED;
    c->pools[layer] = PoolWeights{(const bf16*)w_gate, (const bf16*)w_up, (const bf16*)w_down};
    c->pool_set[layer] = 1;
    tc_destroy(c);     // descriptors are rebuilt lazily
    return MOE_OK;
}

int moe_set_model_weights(moe_ctx* c, int layer, int model, const void* router_w, const float* router_bias,
                          const void* shared_gate_w, const void* ws_gate, const void* ws_up, const void* ws_down,
                          const void* rms_w)
{
    if (!c || !router_w) return MOE_ERR_NULL;
    const moe_config& g = c->cfg;
    if (layer < 0 || layer >= g.n_layers || model < 0 || model >= g.n_models) return MOE_ERR_SHAPE;
    const bool any_shared = ws_gate || ws_up || ws_down;
    if (any_shared && !(ws_gate && ws_up && ws_down)) return MOE_ERR_NULL;
    if (any_shared && g.shared_inter == 0) return MOE_ERR_SHAPE;
    if (!any_shared && g.shared_inter > 0) return MOE_ERR_NULL;
    if (((uintptr_t)router_w | (uintptr_t)shared_gate_w | (uintptr_t)ws_gate | (uintptr_t)ws_up | (uintptr_t)ws_down |
         (uintptr_t)rms_w) & 15)
        return MOE_ERR_SHAPE;
    if (any_shared && tc_supported(c) && !pair_distance_ok(ws_gate, ws_up)) return MOE_ERR_UNSUPPORTED;
    ModelWeights mw{(const bf16*)router_w, router_bias, (const bf16*)shared_gate_w, (const bf16*)ws_gate,
                    (const bf16*)ws_up, (const bf16*)ws_down, (const bf16*)rms_w};
    const size_t i = (size_t)layer * g.n_models + model;
    c->models[i] = mw;
    MOE_CUDA(c, cudaMemcpy(c->d_models + i, &mw, sizeof(mw), cudaMemcpyHostToDevice));
    c->model_set[i] = 1;
    tc_destroy(c);
    route_tc_destroy(c);
    return MOE_OK;
}

int moe_set_slot_table(moe_ctx* c, const int32_t* slot)
{
    if (!c || !slot) return MOE_ERR_NULL;
    const size_t ME = (size_t)c->cfg.n_models * c->cfg.n_experts;
    for (size_t i = 0; i < ME; ++i) if (slot[i] < 0 || slot[i] >= c->cfg.n_slots) return MOE_ERR_SHAPE;
    c->h_slot.assign(slot, slot + ME);
    MOE_CUDA(c, cudaDeviceSynchronize());
    MOE_CUDA(c, cudaMemcpy(c->d_slot, slot, ME * sizeof(int32_t), cudaMemcpyHostToDevice));
    return MOE_OK;
}

int moe_set_tenant_models(moe_ctx* c, const int32_t* model_of_tenant)
{
    if (!c || !model_of_tenant) return MOE_ERR_NULL;
    for (int u = 0; u < c->cfg.n_tenants; ++u)
        if (model_of_tenant[u] < 0 || model_of_tenant[u] >= c->cfg.n_models) return MOE_ERR_SHAPE;
    c->h_model_of_tenant.assign(model_of_tenant, model_of_tenant + c->cfg.n_tenants);
    MOE_CUDA(c, cudaDeviceSynchronize());
    return upload_tenant_tables(c);
}

int moe_form_blocks(const int64_t* load, int n_models, int n_experts, int G, int32_t* block_of_expert)
{
    if (!load || !block_of_expert) return MOE_ERR_NULL;
    if (n_models < 1 || n_experts < 1) return MOE_ERR_SHAPE;
    if (G < 1 || G > n_experts) return MOE_ERR_G;
    const int E = n_experts, B = (E + G - 1) / G;
    std::vector<int> order(E), members(B);
    std::vector<int64_t> weight(B);
    for (int m = 0; m < n_models; ++m) {
        const int64_t* l = load + (size_t)m * E;
        for (int e = 0; e < E; ++e) order[e] = e;
        // heaviest expert first; equal loads in id order
        std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return l[x] > l[y]; });
        std::fill(members.begin(), members.end(), 0);
        std::fill(weight.begin(), weight.end(), (int64_t)0);
        for (int e : order) {
            int best = -1;
            for (int b = 0; b < B; ++b)
                if (members[b] < G && (best < 0 || weight[b] < weight[best])) best = b;
            block_of_expert[(size_t)m * E + e] = best;
            weight[best] += l[e];
            members[best] += 1;
        }
    }
    return MOE_OK;
}

int moe_set_block_table(moe_ctx* c, const int32_t* block_of_expert, int n_blocks)
{
    if (!c) return MOE_ERR_NULL;
    const size_t ME = (size_t)c->cfg.n_models * c->cfg.n_experts;
    MOE_CUDA(c, cudaDeviceSynchronize());
    if (!block_of_expert) {               // back to blocks of G consecutive experts
        if (c->d_block_table) cudaFree(c->d_block_table);
        c->d_block_table = nullptr;
        c->table_blocks = 0;
        return MOE_OK;
    }
    if (n_blocks < 1 || n_blocks > c->cfg.n_experts) return MOE_ERR_SHAPE;
    for (size_t i = 0; i < ME; ++i) if (block_of_expert[i] < 0 || block_of_expert[i] >= n_blocks) return MOE_ERR_SHAPE;
    if (!c->d_block_table) MOE_CUDA(c, dev_alloc(&c->d_block_table, ME));
    MOE_CUDA(c, cudaMemcpy(c->d_block_table, block_of_expert, ME * sizeof(int32_t), cudaMemcpyHostToDevice));
    c->table_blocks = n_blocks;
    return MOE_OK;
}

int moe_residency_enable(moe_ctx* c, int layer, const void* host_gate, const void* host_up, const void* host_down,
                         void* pool_gate, void* pool_up, void* pool_down)
{
    if (!c || !host_gate || !host_up || !host_down || !pool_gate || !pool_up || !pool_down) return MOE_ERR_NULL;
    if (c->cfg.n_layers != 1 || layer != 0) return MOE_ERR_UNSUPPORTED;      // the slot table is one per context
    const int rc = moe_set_expert_pool(c, layer, pool_gate, pool_up, pool_down);
    if (rc != MOE_OK) return rc;
    const size_t ME = (size_t)c->cfg.n_models * c->cfg.n_experts;
    Residency& r = c->res;
    r.h_gate = (const bf16*)host_gate; r.h_up = (const bf16*)host_up; r.h_down = (const bf16*)host_down;
    r.p_gate = (bf16*)pool_gate; r.p_up = (bf16*)pool_up; r.p_down = (bf16*)pool_down;
    r.owner.assign(c->cfg.n_slots, -1);
    r.last_use.assign(c->cfg.n_slots, -1);
    r.slot_of.assign(ME, -1);
    r.clock = 0;
    if (!r.d_active) MOE_CUDA(c, dev_alloc(&r.d_active, ME));
    if (!r.h_active) MOE_CUDA(c, cudaMallocHost((void**)&r.h_active, ME * sizeof(int32_t)));
    r.on = true;
    return MOE_OK;
}

int moe_layer_forward_paged(moe_ctx* c, int layer, const void* x, const int32_t* tenant_id, int T, int G, void* out,
                            int32_t* stats_host, void* stream)
{
    if (!c || !x || !tenant_id || !out) return MOE_ERR_NULL;
    if (!c->res.on || layer != 0) return MOE_ERR_STATE;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x, out)) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, true);
    if (rc != MOE_OK) return rc;
    if (stats_host) stats_host[0] = stats_host[1] = stats_host[2] = stats_host[3] = 0;
    if (T == 0) return MOE_OK;
    const moe_config& g = c->cfg;
    Workspace& w = c->ws;
    Residency& r = c->res;
    cudaStream_t st = (cudaStream_t)stream;
    const int ME = g.n_models * g.n_experts, S = g.n_slots, R = T * g.top_k;
    // 1. the gate, then the set of experts this batch needs, on the host (the one synchronisation of the call)
    MOE_CUDA(c, launch_route(c, layer, (const bf16*)x, tenant_id, T, w.topk_idx, w.topk_w,
                             g.shared_inter > 0 ? w.shared_gate : nullptr, w.tie_flag, st));
    MOE_CUDA(c, cudaMemsetAsync(r.d_active, 0, (size_t)ME * sizeof(int32_t), st));
    mark_active_kernel<<<(R + 255) / 256, 256, 0, st>>>(w.topk_idx, tenant_id, c->d_model_of_tenant, R, g.top_k,
                                                        g.n_experts, g.n_tenants, r.d_active);
    c->launches += 1;
    MOE_CUDA(c, cudaMemcpyAsync(r.h_active, r.d_active, (size_t)ME * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    MOE_CUDA(c, cudaStreamSynchronize(st));
    // 2. residency: hits refresh their slot; every missing expert (ascending id) takes a free slot (lowest index), else
    //    the slot that was used longest ago among those the batch does not need (ties: lowest index)
    r.clock += 1;
    int n_active = 0, hits = 0, loads = 0, evictions = 0;
    for (int i = 0; i < ME; ++i) n_active += r.h_active[i] != 0;
    if (n_active > S) {
        snprintf(c->errbuf, sizeof(c->errbuf), "%d active experts do not fit %d resident slots", n_active, S);
        return MOE_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < ME; ++i)
        if (r.h_active[i] && r.slot_of[i] >= 0) { r.last_use[r.slot_of[i]] = r.clock; ++hits; }
    const size_t wexp = (size_t)g.inter * g.hidden;              // elements of one expert matrix
    for (int i = 0; i < ME; ++i) {
        if (!r.h_active[i] || r.slot_of[i] >= 0) continue;
        int victim = -1;
        for (int s2 = 0; s2 < S && victim < 0; ++s2) if (r.owner[s2] < 0) victim = s2;
        if (victim < 0) {
            for (int s2 = 0; s2 < S; ++s2)
                if (r.last_use[s2] < r.clock && (victim < 0 || r.last_use[s2] < r.last_use[victim])) victim = s2;
            r.slot_of[r.owner[victim]] = -1;
            ++evictions;
        }
        MOE_CUDA(c, cudaMemcpyAsync(r.p_gate + (size_t)victim * wexp, r.h_gate + (size_t)i * wexp, wexp * sizeof(bf16),
                                    cudaMemcpyHostToDevice, st));
        MOE_CUDA(c, cudaMemcpyAsync(r.p_up + (size_t)victim * wexp, r.h_up + (size_t)i * wexp, wexp * sizeof(bf16),
                                    cudaMemcpyHostToDevice, st));
        MOE_CUDA(c, cudaMemcpyAsync(r.p_down + (size_t)victim * wexp, r.h_down + (size_t)i * wexp, wexp * sizeof(bf16),
                                    cudaMemcpyHostToDevice, st));
        r.owner[victim] = i; r.slot_of[i] = victim; r.last_use[victim] = r.clock;
        ++loads;
    }
    for (int i = 0; i < ME; ++i) c->h_slot[i] = r.slot_of[i] >= 0 ? r.slot_of[i] : 0;    // parked experts get no rows
    MOE_CUDA(c, cudaMemcpyAsync(c->d_slot, c->h_slot.data(), (size_t)ME * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    if (stats_host) { stats_host[0] = n_active; stats_host[1] = hits; stats_host[2] = loads; stats_host[3] = evictions; }
    // 3. the rest of the layer on the routing results that are already in the workspace
    return layer_forward_impl(c, layer, (const bf16*)x, tenant_id, T, G, nullptr, (bf16*)out, st, true);
}

int moe_set_option(moe_ctx* c, int option, int value)
{
    if (!c) return MOE_ERR_NULL;
    if (option == MOE_OPT_EXPERT_PATH) {
        if (value < MOE_PATH_AUTO || value > MOE_PATH_TCGEN05) return MOE_ERR_SHAPE;
        if (value == MOE_PATH_TCGEN05 && !tc_supported(c)) return MOE_ERR_UNSUPPORTED;
        c->expert_path = value;
        return MOE_OK;
    }
    if (option == MOE_OPT_PAIR_MODE) {
        if (value < 0 || value > 2) return MOE_ERR_SHAPE;
        c->pair_mode_enabled = value;
        return MOE_OK;
    }
    if (option == MOE_OPT_ROUTE_LANES) {
        if (value < 1 || value > 2) return MOE_ERR_SHAPE;
        c->route_lanes2 = value == 2 ? 1 : 0;
        return MOE_OK;
    }
    if (option == MOE_OPT_EARLY_SHARED) {
        if (value < 0 || value > 2) return MOE_ERR_SHAPE;
        c->early_shared_enabled = value;
        return MOE_OK;
    }
    if (option == MOE_OPT_EARLY_SHARED_SMS) {
        if (value < 2) return MOE_ERR_SHAPE;
        c->early_shared_sms = value & ~1;
        return MOE_OK;
    }
    if (option == MOE_OPT_TOKEN_MAJOR) {
        c->token_major_enabled = value ? 1 : 0;
        return MOE_OK;
    }
    if (option == MOE_OPT_WIDE_TILES) {
        if (value < 0 || value > 2) return MOE_ERR_SHAPE;
        c->wide_tiles_enabled = value;
        return MOE_OK;
    }
    if (option == MOE_OPT_BACKGROUND_LANES) {
        if (value < 0 || value > 2) return MOE_ERR_SHAPE;
        c->background_enabled = value;
        return MOE_OK;
    }
    if (option == MOE_OPT_HEAD_UNITS) {
        c->head_units_enabled = value ? 1 : 0;
        return MOE_OK;
    }
    if (option == MOE_OPT_FUSED_DISPATCH) {
        c->fused_dispatch_enabled = value ? 1 : 0;
        return MOE_OK;
    }
    if (option == MOE_OPT_DISPATCH_MODE) {
        if (value != MOE_DISPATCH_SHARED && value != MOE_DISPATCH_PRIVATE) return MOE_ERR_SHAPE;
        c->dispatch_private = value == MOE_DISPATCH_PRIVATE ? 1 : 0;
        return MOE_OK;
    }
    if (option == MOE_OPT_ROUTE_PATH) {
        if (value < MOE_PATH_AUTO || value > MOE_PATH_TCGEN05) return MOE_ERR_SHAPE;
        if (value == MOE_PATH_TCGEN05 && !route_tc_supported(c)) return MOE_ERR_UNSUPPORTED;
        c->route_path = value;
        return MOE_OK;
    }
    return MOE_ERR_SHAPE;
}

int moe_route(moe_ctx* c, int layer, const void* x, const int32_t* tenant_id, int T, int32_t* topk_idx, float* topk_w,
              float* shared_gate, uint8_t* tie_flag, void* stream)
{
    if (!c || !x || !tenant_id || !topk_idx || !topk_w) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x)) return MOE_ERR_SHAPE;
    const int rc = check_layer_ready(c, layer, false, false);
    if (rc != MOE_OK) return rc;
    if (T == 0) return MOE_OK;
    MOE_CUDA(c, launch_route(c, layer, (const bf16*)x, tenant_id, T, topk_idx, topk_w, shared_gate, tie_flag,
                             (cudaStream_t)stream));
    return MOE_OK;
}

int moe_dispatch(moe_ctx* c, const void* x, const int32_t* topk_idx, const int32_t* tenant_id, int T, int G,
                 int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off,
                 int32_t* group_off, void* x_perm, void* stream)
{
    if (!c || !topk_idx || !tenant_id || !perm || !inv_perm || !expert_off) return MOE_ERR_NULL;
    if (x_perm && !x) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x, x_perm)) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    if (T == 0) return MOE_OK;
    MOE_CUDA(c, launch_dispatch(c, (const bf16*)x, topk_idx, tenant_id, T, G, perm, inv_perm, tenant_expert_count,
                                expert_off, group_off, (bf16*)x_perm, (cudaStream_t)stream));
    return MOE_OK;
}

int moe_experts(moe_ctx* c, int layer, const void* x, const void* x_perm, const int32_t* perm, const int32_t* expert_off,
                const int32_t* tenant_id, int T, int G, float* y_perm, float* y_shared, void* stream)
{
    if (!c || !x_perm || !expert_off || !y_perm) return MOE_ERR_NULL;
    if (y_shared && (!x || !tenant_id)) return MOE_ERR_NULL;
    if (misaligned16(x_perm, x, y_perm, y_shared)) return MOE_ERR_SHAPE;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, y_shared != nullptr);
    if (rc != MOE_OK) return rc;
    if (T == 0) return MOE_OK;
    // reading the tokens in place needs x and perm; without them the permuted copy is used
    return experts_impl(c, layer, (const bf16*)x, (const bf16*)x_perm, x ? perm : nullptr, expert_off, tenant_id, T, G,
                        (float*)y_perm, (float*)y_shared, (cudaStream_t)stream);
}

int moe_combine(moe_ctx* c, const float* y_perm, const int32_t* inv_perm, const float* topk_w, const float* y_shared,
                const float* shared_gate, int T, void* out, void* stream)
{
    if (!c || !y_perm || !inv_perm || !topk_w || !out) return MOE_ERR_NULL;
    if ((y_shared == nullptr) != (shared_gate == nullptr)) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(y_perm, y_shared, out)) return MOE_ERR_SHAPE;
    if (T == 0) return MOE_OK;
    MOE_CUDA(c, launch_combine(c, (const float*)y_perm, inv_perm, topk_w, (const float*)y_shared, shared_gate, nullptr,
                               T, (bf16*)out, (cudaStream_t)stream));
    return MOE_OK;
}

int moe_layer_forward(moe_ctx* c, int layer, const void* x, const int32_t* tenant_id, int T, int G, void* out,
                      void* stream)
{
    if (!c || !x || !tenant_id || !out) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x, out)) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, true);
    if (rc != MOE_OK) return rc;
    if (T == 0) return MOE_OK;
    return layer_forward_impl(c, layer, (const bf16*)x, tenant_id, T, G, nullptr, (bf16*)out, (cudaStream_t)stream);
}

int moe_layer_forward_host(moe_ctx* c, int layer, const void* x_host, const int32_t* tenant_id_host, int T, int G,
                           void* out_host, void* stream)
{
    if (!c || !x_host || !tenant_id_host || !out_host) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, true);
    if (rc != MOE_OK) return rc;
    if (T == 0) return MOE_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t xbytes = (size_t)T * c->cfg.hidden * sizeof(bf16);
    MOE_CUDA(c, cudaMemcpyAsync(c->ws.x_stage, x_host, xbytes, cudaMemcpyHostToDevice, st));
    MOE_CUDA(c, cudaMemcpyAsync(c->ws.tenant_stage, tenant_id_host, (size_t)T * sizeof(int32_t),
                                cudaMemcpyHostToDevice, st));
    const int rc2 = layer_forward_impl(c, layer, c->ws.x_stage, c->ws.tenant_stage, T, G, nullptr, c->ws.out_stage, st);
    if (rc2 != MOE_OK) return rc2;
    MOE_CUDA(c, cudaMemcpyAsync(out_host, c->ws.out_stage, xbytes, cudaMemcpyDeviceToHost, st));
    MOE_CUDA(c, cudaStreamSynchronize(st));
    return MOE_OK;
}

int moe_layer_forward_host_submit(moe_ctx* c, int layer, const void* x_host, const int32_t* tenant_id_host, int T, int G,
                                  void* out_host, void* stream, int64_t* ticket)
{
    if (!c || !x_host || !tenant_id_host || !out_host || !ticket) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, true);
    if (rc != MOE_OK) return rc;
    const int64_t n = c->submitted;
    const int slot = (int)(n & 1);
    // the slot's previous user (two submissions ago) must have delivered its outputs before its buffers are reused
    if (n >= 2 && c->waited[slot] < n - 2) {
        MOE_CUDA(c, cudaEventSynchronize(c->ev_out[slot]));
        c->waited[slot] = n - 2;
    }
    cudaStream_t st = (cudaStream_t)stream;
    bf16* xs = slot ? c->ws.x_stage2 : c->ws.x_stage;
    int32_t* ts = slot ? c->ws.tenant_stage2 : c->ws.tenant_stage;
    bf16* os = slot ? c->ws.out_stage2 : c->ws.out_stage;
    const size_t xbytes = (size_t)T * c->cfg.hidden * sizeof(bf16);
    if (T > 0) {
        // inputs on the copy-in stream (beside the layer pass of the submission before), the layer on the caller's
        // stream, outputs on the copy-out stream (beside the next layer pass)
        MOE_CUDA(c, cudaMemcpyAsync(xs, x_host, xbytes, cudaMemcpyHostToDevice, c->copy_in));
        MOE_CUDA(c, cudaMemcpyAsync(ts, tenant_id_host, (size_t)T * sizeof(int32_t), cudaMemcpyHostToDevice, c->copy_in));
        MOE_CUDA(c, cudaEventRecord(c->ev_in[slot], c->copy_in));
        MOE_CUDA(c, cudaStreamWaitEvent(st, c->ev_in[slot], 0));
        const int rc2 = layer_forward_impl(c, layer, xs, ts, T, G, nullptr, os, st);
        if (rc2 != MOE_OK) return rc2;
        MOE_CUDA(c, cudaEventRecord(c->ev_done[slot], st));
        MOE_CUDA(c, cudaStreamWaitEvent(c->copy_out, c->ev_done[slot], 0));
        MOE_CUDA(c, cudaMemcpyAsync(out_host, os, xbytes, cudaMemcpyDeviceToHost, c->copy_out));
    }
    MOE_CUDA(c, cudaEventRecord(c->ev_out[slot], c->copy_out));
    *ticket = n;
    c->submitted = n + 1;
    return MOE_OK;
}

int moe_layer_forward_host_wait(moe_ctx* c, int64_t ticket)
{
    if (!c) return MOE_ERR_NULL;
    if (ticket < 0 || ticket >= c->submitted) return MOE_ERR_SHAPE;
    const int slot = (int)(ticket & 1);
    if (c->waited[slot] >= ticket) return MOE_OK;                   // already known to be complete
    if (ticket + 2 < c->submitted) return MOE_OK;                   // its slot has been reused: that submit waited for it
    MOE_CUDA(c, cudaEventSynchronize(c->ev_out[slot]));
    c->waited[slot] = ticket;
    return MOE_OK;
}

int moe_layer_forward_timed(moe_ctx* c, int layer, const void* x, const int32_t* tenant_id, int T, int G, void* out,
                            float* stage_ms_host, void* stream)
{
    if (!c || !x || !tenant_id || !out || !stage_ms_host) return MOE_ERR_NULL;
    if (T < 1 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x, out)) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    const int rc = check_layer_ready(c, layer, true, true);
    if (rc != MOE_OK) return rc;
    for (int i = 0; i < kEvCount; ++i)
        if (!c->ev[i]) MOE_CUDA(c, cudaEventCreate(&c->ev[i]));
    c->timing = true;
    const int rc2 = layer_forward_impl(c, layer, (const bf16*)x, tenant_id, T, G, nullptr, (bf16*)out,
                                       (cudaStream_t)stream);
    c->timing = false;
    if (rc2 != MOE_OK) return rc2;
    MOE_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
    for (int i = 1; i < kEvCount; ++i) MOE_CUDA(c, cudaEventElapsedTime(&stage_ms_host[i - 1], c->ev[i - 1], c->ev[i]));
    return MOE_OK;
}

int moe_stack_forward(moe_ctx* c, void* x_inout, const int32_t* tenant_id, int T, int G, void* dbg_layer_inputs,
                      void* dbg_layer_outputs, void* stream)
{
    if (!c || !x_inout || !tenant_id) return MOE_ERR_NULL;
    if (T < 0 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    if (misaligned16(x_inout, dbg_layer_inputs, dbg_layer_outputs)) return MOE_ERR_SHAPE;
    if (G < 1 || G > c->cfg.n_experts) return MOE_ERR_G;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        const int rc = check_layer_ready(c, l, true, true);
        if (rc != MOE_OK) return rc;
        for (int m = 0; m < c->cfg.n_models; ++m)
            if (!c->models[(size_t)l * c->cfg.n_models + m].rms_w) return MOE_ERR_STATE;
    }
    if (T == 0) return MOE_OK;
    cudaStream_t st = (cudaStream_t)stream;
    bf16* x = (bf16*)x_inout;
    const size_t n = (size_t)T * c->cfg.hidden;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        bf16* xn = dbg_layer_inputs ? (bf16*)dbg_layer_inputs + (size_t)l * n : c->ws.xn;
        MOE_CUDA(c, launch_rmsnorm(c, l, x, tenant_id, T, xn, st));
        const int rc = layer_forward_impl(c, l, xn, tenant_id, T, G, x, x, st);
        if (rc != MOE_OK) return rc;
        if (dbg_layer_outputs)
            MOE_CUDA(c, cudaMemcpyAsync((bf16*)dbg_layer_outputs + (size_t)l * n, x, n * sizeof(bf16),
                                        cudaMemcpyDeviceToDevice, st));
    }
    return MOE_OK;
}

int moe_get_workspace(moe_ctx* c, int32_t** topk_idx, float** topk_w, float** shared_gate, uint8_t** tie_flag,
                      int32_t** perm, int32_t** inv_perm, int32_t** expert_off, int32_t** group_off)
{
    if (!c) return MOE_ERR_NULL;
    if (topk_idx) *topk_idx = c->ws.topk_idx;
    if (topk_w) *topk_w = c->ws.topk_w;
    if (shared_gate) *shared_gate = c->ws.shared_gate;
    if (tie_flag) *tie_flag = c->ws.tie_flag;
    if (perm) *perm = c->ws.perm;
    if (inv_perm) *inv_perm = c->ws.inv_perm;
    if (expert_off) *expert_off = c->ws.expert_off;
    if (group_off) *group_off = c->ws.group_off;
    return MOE_OK;
}

int moe_last_status(moe_ctx* c, int32_t* status_host, int32_t* stats_host)
{
    if (!c || !status_host) return MOE_ERR_NULL;
    MOE_CUDA(c, cudaDeviceSynchronize());
    MOE_CUDA(c, cudaMemcpy(status_host, c->ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (stats_host) MOE_CUDA(c, cudaMemcpy(stats_host, c->ws.stats, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost));
    MOE_CUDA(c, cudaMemset(c->ws.status, 0, sizeof(int32_t)));
    return MOE_OK;
}

int moe_last_plan(moe_ctx* c, int T, int32_t* plan_host)
{
    if (!c || !plan_host) return MOE_ERR_NULL;
    if (T < 1 || T > c->cfg.max_tokens) return MOE_ERR_SHAPE;
    MOE_CUDA(c, cudaDeviceSynchronize());
    MOE_CUDA(c, cudaMemcpy(plan_host, c->ws.plan_counts, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost));
    plan_host[2] = make_plan_args(c, T, 1, false).tile_rows;
    return MOE_OK;
}

int64_t moe_launch_count(moe_ctx* c) { return c ? c->launches : -1; }

const char* moe_strerror(int status)
{
    switch (status) {
        case MOE_OK: return "ok";
        case MOE_ERR_NULL: return "a required pointer is NULL";
        case MOE_ERR_SHAPE: return "a size or id is out of range";
        case MOE_ERR_G: return "G must be in [1, n_experts]";
        case MOE_ERR_STATE: return "weights of the requested layer/model were not set";
        case MOE_ERR_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "a CUDA call failed";
        case MOE_ERR_ALLOC: return "workspace allocation failed";
        case MOE_ERR_UNSUPPORTED: return "shape not supported by the kernels";
        default: return "unknown status";
    }
}

}  // extern "C"
