// Routing requests batched per expert block: per-(tenant, expert) histogram, prefix scan, stable ranks,
// token permute into expert segments (paper Sec. 3: the orchestrator groups the routed tokens into one
// request per block; Sec. 4.1: whatever goes to the same block travels in one invocation).  Rows are
// ordered by (model, expert, tenant, token); the order is produced without order-dependent atomics so
// that the permutation is reproducible bit for bit.  The invocation statistics follow the orchestrator
// placement (Sec. 4.2, Sec. 5): a shared orchestrator sends one invocation per non-empty block, private
// orchestrators one per (tenant, block) pair that has rows.
#include <cstring>
#include <mutex>

#include "internal.h"
#include "dispatch_small.cuh"
#include "plan.cuh"
#include "scan.cuh"

namespace faasmoe {

namespace {

// D1 (large batches): every block ranks the rows of its chunk.  One warp walks the chunk in row order; rows
// that share a bin inside one step are ranked by lane order (= row order), so the rank of a row inside
// (block, bin) does not depend on timing.  The pair (bin, rank in block) is parked in inv_perm[r] for D2.
// The block that finishes last turns the per-block counts into offsets: totals per bin, exclusive scan in key
// order, per-block bases, the offset tables the caller sees, and (optionally) the expert work plan.
constexpr int kCountThreads = 512;

__global__ void __launch_bounds__(kCountThreads)
dispatch_count_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ tenant_id, int nblk, int nbins,
                      int R, int k, int E, int M, int G, int n_tenants, BinMap bm, int32_t* __restrict__ block_cnt,
                      int32_t* __restrict__ bin_off, int32_t* __restrict__ inv_perm,
                      int32_t* __restrict__ tenant_expert_count, int32_t* __restrict__ expert_off,
                      int32_t* __restrict__ group_off, int32_t* __restrict__ stats, int32_t* __restrict__ status,
                      int32_t* __restrict__ done_counter, int do_plan, PlanArgs pa, int private_mode,
                      const int32_t* __restrict__ block_table, int table_blocks)
{
    extern __shared__ int32_t s_tot[];       // [nbins] counts of this block; in the last block: totals, then offsets,
                                             // followed by the plan's scratch
    __shared__ int32_t s_part[33];
    __shared__ int32_t s_count[2];
    __shared__ int s_last;
    pdl_wait();
    pdl_launch_dependents();
    const int tid = threadIdx.x, nth = blockDim.x, lane = tid & 31, warp = tid >> 5;
    // every thread looks up the bin of one row of the chunk (the lookups are chains of dependent loads: all of them
    // in flight at once), then one warp walks the bins in row order out of shared memory
    __shared__ unsigned short s_bin[kDispatchChunk];
    const int r0 = blockIdx.x * kDispatchChunk;
    const int r1 = min(R, r0 + kDispatchChunk);
    for (int b = tid; b < nbins; b += nth) s_tot[b] = 0;
    for (int r = r0 + tid; r < r1; r += nth) s_bin[r - r0] = (unsigned short)row_bin(bm, tenant_id[r / k], topk_idx[r], status);
    __syncthreads();
    if (warp == 0) {
        for (int rr = r0; rr < r1; rr += 32) {
            const int r = rr + lane;
            const bool live = r < r1;
            int bin = -1 - lane;                 // distinct dummy keys for idle lanes
            if (live) bin = s_bin[r - r0];
            const unsigned peers = __match_any_sync(0xffffffffu, bin);
            const int leader = __ffs(peers) - 1;
            const int rank = __popc(peers & ((1u << lane) - 1u));
            int start = 0;
            if (live && lane == leader) { start = s_tot[bin]; s_tot[bin] = start + __popc(peers); }
            start = __shfl_sync(0xffffffffu, start, leader);
            if (live) inv_perm[r] = bin | ((start + rank) << 16);      // bin < 8192, rank < kDispatchChunk
            __syncwarp();
        }
    }
    __syncthreads();
    int32_t* mine = block_cnt + (size_t)blockIdx.x * nbins;
    for (int b = tid; b < nbins; b += nth) mine[b] = s_tot[b];
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(done_counter, 1) == nblk - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) *done_counter = 0;             // ready for the next call on this stream
    // totals per bin; block_cnt becomes the exclusive prefix over blocks.  One thread per bin (neighbouring
    // threads read neighbouring counters); the counts of 16 blocks are fetched before any is replaced, so the
    // loads of a round are in flight together.
    for (int b = tid; b < nbins; b += nth) {
        int run = 0;
        for (int blk0 = 0; blk0 < nblk; blk0 += 16) {
            int cnt[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) cnt[j] = blk0 + j < nblk ? __ldcg(block_cnt + (size_t)(blk0 + j) * nbins + b) : 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (blk0 + j < nblk) block_cnt[(size_t)(blk0 + j) * nbins + b] = run;
                run += cnt[j];
            }
        }
        s_tot[b] = run;
    }
    __syncthreads();
    scan_and_tables(s_tot, s_part, s_count, nbins, R, E, M, G, n_tenants, bm, bin_off, tenant_expert_count,
                    expert_off, group_off, stats, private_mode, block_table, table_blocks);
    if (do_plan) {
        __syncthreads();
        plan_body(expert_off, pa, s_tot + nbins, s_part);
    }
}

// D2 (large batches): position of every row = offset of its bin + rows of that bin in earlier blocks + rank in
// its block; writes perm / inv_perm and, with GATHER, copies the token's row to its place in x_perm (one warp
// per row, 16-byte vectors).
template <bool GATHER>
__global__ void __launch_bounds__(256)
dispatch_place_kernel(int R, int k, int nbins, const int32_t* __restrict__ block_cnt, const int32_t* __restrict__ bin_off,
                      int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, const bf16* __restrict__ x,
                      bf16* __restrict__ x_perm, int H, const int32_t* __restrict__ expert_off, int do_plan, PlanArgs pa)
{
    pdl_wait();
    pdl_launch_dependents();
    if (do_plan && blockIdx.x == gridDim.x - 1) {
        // one extra block builds the expert work plan (it needs the offset tables of the counting kernel only) while
        // the other blocks place and copy the rows: the plan is off the tail of the counting kernel's last block
        extern __shared__ int32_t s_plan[];
        __shared__ int32_t s_part[33];
        plan_body(expert_off, pa, s_plan, s_part);
        return;
    }
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
    const int r = GATHER ? gtid >> 5 : gtid;
    if (r >= R) return;
    const int lane = threadIdx.x & 31;
    const int packed = inv_perm[r];
    const int bin = packed & 0xffff, lrank = packed >> 16;
    const int pos = bin_off[bin] + block_cnt[(size_t)(r / kDispatchChunk) * nbins + bin] + lrank;
    if (GATHER) {
        __syncwarp();                            // every lane has read the parked value before lane 0 replaces it
        if (lane == 0) { perm[pos] = r; inv_perm[r] = pos; }
        const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)(r / k) * H);
        uint4* dst = reinterpret_cast<uint4*>(x_perm + (size_t)pos * H);
        for (int v = lane; v < (H >> 3); v += 32) dst[v] = src[v];
    } else {
        perm[pos] = r;
        inv_perm[r] = pos;
    }
}

// Small batches: the whole dispatch in one block (dispatch_small.cuh).
constexpr int kSmallRows = 2048;   // above this the serial ranking pass of one warp costs more than the extra launches

__global__ void __launch_bounds__(1024, 1)
dispatch_small_kernel(const __grid_constant__ SmallDispatchArgs a)
{
    extern __shared__ int32_t s_tot[];       // [nbins], then the plan's scratch, then the bin of every row (u16)
    pdl_wait();
    pdl_launch_dependents();
    dispatch_small_body(a, s_tot);
}

// D4: x_perm[pos] = x[perm[pos] / k].  One warp per row, 16-byte vectors.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const bf16* __restrict__ x, const int32_t* __restrict__ perm, int R, int k, int H,
                   bf16* __restrict__ x_perm)
{
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= R) return;
    const int t = perm[warp] / k;
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * H);
    uint4* dst = reinterpret_cast<uint4*>(x_perm + (size_t)warp * H);
    for (int v = lane; v < (H >> 3); v += 32) dst[v] = src[v];
}

// Token sort by (model, token) for the shared experts of a multi-model pool.
__global__ void __launch_bounds__(32)
token_hist_kernel(const int32_t* __restrict__ tenant_id, int T, int n_tenants, int M,
                  const int32_t* __restrict__ model_of_tenant, int32_t* __restrict__ tok_block_cnt)
{
    __shared__ int32_t s_cnt[kMaxExperts];
    for (int m = threadIdx.x; m < M; m += 32) s_cnt[m] = 0;
    __syncwarp();
    const int t0 = blockIdx.x * kDispatchChunk, t1 = min(T, t0 + kDispatchChunk);
    for (int t = t0 + threadIdx.x; t < t1; t += 32) {
        int u = tenant_id[t];
        if (u < 0 || u >= n_tenants) u = 0;
        atomicAdd(&s_cnt[model_of_tenant[u]], 1);
    }
    __syncwarp();
    for (int m = threadIdx.x; m < M; m += 32) tok_block_cnt[(size_t)blockIdx.x * M + m] = s_cnt[m];
}

__global__ void __launch_bounds__(256)
token_scan_kernel(int nblk, int M, int T, int32_t* __restrict__ tok_block_cnt, int32_t* __restrict__ model_tok_off)
{
    __shared__ int32_t s_tot[kMaxExperts];
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
        int run = 0;
        for (int blk = 0; blk < nblk; ++blk) {
            const int c = tok_block_cnt[(size_t)blk * M + m];
            tok_block_cnt[(size_t)blk * M + m] = run;
            run += c;
        }
        s_tot[m] = run;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int m = 0; m < M; ++m) { model_tok_off[m] = run; run += s_tot[m]; }
        model_tok_off[M] = run;
    }
}

__global__ void __launch_bounds__(32)
token_rank_kernel(const int32_t* __restrict__ tenant_id, int T, int n_tenants, int M,
                  const int32_t* __restrict__ model_of_tenant, const int32_t* __restrict__ tok_block_cnt,
                  const int32_t* __restrict__ model_tok_off, int32_t* __restrict__ tok_perm,
                  int32_t* __restrict__ tok_inv)
{
    __shared__ int32_t s_next[kMaxExperts];
    const int lane = threadIdx.x;
    for (int m = lane; m < M; m += 32) s_next[m] = model_tok_off[m] + tok_block_cnt[(size_t)blockIdx.x * M + m];
    __syncwarp();
    const int t0 = blockIdx.x * kDispatchChunk, t1 = min(T, t0 + kDispatchChunk);
    for (int tt = t0; tt < t1; tt += 32) {
        const int t = tt + lane;
        const bool live = t < t1;
        int key = -1 - lane;
        if (live) {
            int u = tenant_id[t];
            if (u < 0 || u >= n_tenants) u = 0;
            key = model_of_tenant[u];
        }
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        const int leader = __ffs(peers) - 1;
        const int rank = __popc(peers & ((1u << lane) - 1u));
        int start = 0;
        if (live && lane == leader) { start = s_next[key]; s_next[key] = start + __popc(peers); }
        start = __shfl_sync(0xffffffffu, start, leader);
        if (live) { tok_perm[start + rank] = t; tok_inv[t] = start + rank; }
        __syncwarp();
    }
}

BinMap make_binmap(const moe_ctx* c)
{
    BinMap bm;
    bm.model_of_tenant = c->d_model_of_tenant;
    bm.tenant_local = c->d_tenant_local;
    bm.bin_base = c->d_bin_base;
    bm.tenants_in_model = c->d_tenants_in_model;
    bm.n_tenants = c->cfg.n_tenants;
    bm.E = c->cfg.n_experts;
    return bm;
}

// Arguments of the one-block dispatch for a batch of at most kSmallRows rows.
void small_dispatch_args(moe_ctx* c, const bf16* x, const int32_t* topk_idx, const int32_t* tenant_id, int T, int G,
                         int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off,
                         int32_t* group_off, bf16* x_perm, bool with_plan, bool plan_shared, SmallDispatchArgs* out,
                         size_t* smem_bytes, bool* gather_inside)
{
    const moe_config& g = c->cfg;
    const int k = g.top_k, R = T * k, nbins = c->nbins;
    SmallDispatchArgs& a = *out;
    memset(&a, 0, sizeof(a));
    // the gather rides along while it is small
    *gather_inside = x_perm && (size_t)R * g.hidden * sizeof(bf16) <= (1u << 20);
    // the expert work plan rides along when the shared-expert tiles need no token sort (one model)
    const bool do_plan = with_plan && g.n_models == 1;
    size_t plan_ints = 0;
    if (do_plan) { a.pa = make_plan_args(c, T, G, plan_shared); plan_ints = plan_smem_ints(c, G); }
    a.topk_idx = topk_idx; a.tenant_id = tenant_id; a.R = R; a.k = k; a.bm = make_binmap(c); a.nbins = nbins;
    a.E = g.n_experts; a.M = g.n_models; a.G = G; a.n_tenants = g.n_tenants;
    a.perm = perm; a.inv_perm = inv_perm; a.tenant_expert_count = tenant_expert_count; a.expert_off = expert_off;
    a.group_off = group_off; a.stats = c->ws.stats; a.status = c->ws.status;
    a.x = x; a.x_perm = *gather_inside ? x_perm : nullptr; a.H = g.hidden;
    a.do_plan = do_plan ? 1 : 0; a.plan_ints = (int)plan_ints;
    a.bin_off = c->dispatch_private ? c->ws.bin_off : nullptr; a.private_mode = c->dispatch_private;
    a.block_table = c->d_block_table; a.table_blocks = c->table_blocks;
    *smem_bytes = (size_t)nbins * sizeof(int32_t) + plan_ints * sizeof(int32_t) + (((size_t)R * 2 + 15) & ~(size_t)15);
}

}  // namespace

cudaError_t launch_route_dispatch(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int G,
                                  int32_t* topk_idx, float* topk_w, float* shared_gate, uint8_t* tie_flag, int32_t* perm,
                                  int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off, int32_t* group_off,
                                  bf16* x_perm, cudaStream_t st, bool plan_shared, bool* fused, bool* plan_done)
{
    *fused = false;
    *plan_done = false;
    const moe_config& g = c->cfg;
    const bool tc = c->route_path != MOE_PATH_FMA && route_tc_supported(c);
    // One CTA routes the batch (at most 128 tokens of one model): it holds every routed row when its top-k step ends
    // and goes on to the dispatch and the plan -- one launch and one round trip through global memory fewer on the
    // latency chain of a small batch.
    if (tc && c->fused_dispatch_enabled && T <= kFusedDispatchTokens && g.n_models == 1 && T * g.top_k <= kSmallRows) {
        SmallDispatchArgs a;
        size_t smem_small = 0;
        bool gather_inside = false;
        small_dispatch_args(c, x, topk_idx, tenant_id, T, G, perm, inv_perm, tenant_expert_count, expert_off, group_off,
                            x_perm, true, plan_shared, &a, &smem_small, &gather_inside);
        if (smem_small <= kFusedDispatchSmem) {
            const cudaError_t e = launch_route_tc(c, layer, x, tenant_id, T, topk_idx, topk_w, shared_gate, tie_flag, st,
                                                  &a, smem_small);
            if (e != cudaSuccess) return e;
            *fused = true;
            *plan_done = a.do_plan != 0;
            if (x_perm && !gather_inside) {
                // (more rows than one block should copy: the permuted copy is made by a grid of its own)
                gather_rows_kernel<<<(T * g.top_k * 32 + 255) / 256, 256, 0, st>>>(x, perm, T * g.top_k, g.top_k, g.hidden, x_perm);
                c->launches += 1;
                return cudaGetLastError();
            }
            return cudaSuccess;
        }
    }
    return launch_route(c, layer, x, tenant_id, T, topk_idx, topk_w, shared_gate, tie_flag, st);
}

cudaError_t launch_dispatch(moe_ctx* c, const bf16* x, const int32_t* topk_idx, const int32_t* tenant_id, int T, int G,
                            int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off,
                            int32_t* group_off, bf16* x_perm, cudaStream_t st, bool with_plan, bool plan_shared,
                            bool* plan_done)
{
    if (plan_done) *plan_done = false;
    const moe_config& g = c->cfg;
    const int k = g.top_k, R = T * k;
    const int nblk = (R + kDispatchChunk - 1) / kDispatchChunk;
    const int nbins = c->nbins;
    const BinMap bm = make_binmap(c);
    const size_t smem = (size_t)nbins * sizeof(int32_t);
    if (R <= kSmallRows) {
        // few rows: one block does everything
        SmallDispatchArgs a;
        size_t smem_small = 0;
        bool gather_inside = false;
        small_dispatch_args(c, x, topk_idx, tenant_id, T, G, perm, inv_perm, tenant_expert_count, expert_off, group_off,
                            x_perm, with_plan, plan_shared, &a, &smem_small, &gather_inside);
        const int threads = (R <= 512 && nbins <= 1024) ? 256 : 1024;
        if (smem_small > 48 * 1024)
            cudaFuncSetAttribute(dispatch_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_small);
        launch_pdl(dispatch_small_kernel, dim3(1), dim3(threads), smem_small, st, a);
        if (plan_done) *plan_done = a.do_plan != 0;
        c->launches += 1;
        if (x_perm && !gather_inside) {
            gather_rows_kernel<<<(R * 32 + 255) / 256, 256, 0, st>>>(x, perm, R, k, g.hidden, x_perm);
            c->launches += 1;
        }
        return cudaGetLastError();
    }
    const bool do_plan = with_plan && g.n_models == 1;
    PlanArgs pa;
    memset(&pa, 0, sizeof(pa));
    size_t plan_ints = 0;
    if (do_plan) { pa = make_plan_args(c, T, G, plan_shared); plan_ints = plan_smem_ints(c, G); }
    // the plan rides in an extra block of the placing kernel when its scratch fits the default shared memory
    const bool plan_in_place = do_plan && plan_ints * sizeof(int32_t) <= 40 * 1024;
    const bool plan_in_count = do_plan && !plan_in_place;
    const size_t smem_count = smem + (plan_in_count ? plan_ints : 0) * sizeof(int32_t);
    if (smem_count > 48 * 1024)
        cudaFuncSetAttribute(dispatch_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_count);
    const size_t smem_place = plan_in_place ? plan_ints * sizeof(int32_t) : 0;
    launch_pdl(dispatch_count_kernel, dim3(nblk), dim3(kCountThreads), smem_count, st,
        topk_idx, tenant_id, nblk, nbins, R, k, g.n_experts, g.n_models, G, g.n_tenants, bm, c->ws.block_cnt, c->ws.bin_off,
        inv_perm, tenant_expert_count, expert_off, group_off, c->ws.stats, c->ws.status, c->ws.dispatch_done,
        plan_in_count ? 1 : 0, pa, c->dispatch_private, c->d_block_table, c->table_blocks);
    if (plan_done) *plan_done = do_plan;
    const unsigned extra = plan_in_place ? 1u : 0u;
    if (x_perm)
        launch_pdl(dispatch_place_kernel<true>, dim3((R * 32 + 255) / 256 + extra), dim3(256), smem_place, st, R, k, nbins,
                   c->ws.block_cnt, c->ws.bin_off, perm, inv_perm, x, x_perm, g.hidden, expert_off, plan_in_place ? 1 : 0, pa);
    else
        launch_pdl(dispatch_place_kernel<false>, dim3((R + 255) / 256 + extra), dim3(256), smem_place, st, R, k, nbins,
                   c->ws.block_cnt, c->ws.bin_off, perm, inv_perm, nullptr, nullptr, g.hidden, expert_off, plan_in_place ? 1 : 0, pa);
    c->launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_token_sort(moe_ctx* c, const bf16* x, const int32_t* tenant_id, int T, cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const int nblk = (T + kDispatchChunk - 1) / kDispatchChunk;
    token_hist_kernel<<<nblk, 32, 0, st>>>(tenant_id, T, g.n_tenants, g.n_models, c->d_model_of_tenant,
                                           c->ws.tok_block_cnt);
    token_scan_kernel<<<1, 256, 0, st>>>(nblk, g.n_models, T, c->ws.tok_block_cnt, c->ws.model_tok_off);
    token_rank_kernel<<<nblk, 32, 0, st>>>(tenant_id, T, g.n_tenants, g.n_models, c->d_model_of_tenant,
                                           c->ws.tok_block_cnt, c->ws.model_tok_off, c->ws.tok_perm, c->ws.tok_inv);
    const int blocks = (T * 32 + 255) / 256;
    gather_rows_kernel<<<blocks, 256, 0, st>>>(x, c->ws.tok_perm, T, 1, g.hidden, c->ws.xs_perm);
    c->launches += 4;
    return cudaGetLastError();
}

}  // namespace faasmoe


// ---------------------------------------------------------------------------------------------
// Dispatch without any allocation.
//
// Some callers may not allocate device memory: a plug-in that runs inside a host application
// whose memory pool is fixed at start-up, code on a latency-critical path where cudaMalloc's
// implicit device synchronisation is not acceptable, or a process that has been told to stay
// inside a memory budget it already spent.  Such callers cannot create a moe_ctx either, because
// moe_create allocates the workspace.  For them the scratch of the dispatch kernels (per-block
// histograms, bin offsets, the tenant tables derived from model_of_tenant, the statistics and
// the status word) lives in the fixed array below, which every GPU that loads this library
// holds until the process exits.
// ---------------------------------------------------------------------------------------------

namespace faasmoe {
namespace {

constexpr int kNoAllocWords = MOE_DISPATCH_NOALLOC_MAX_WORDS;
static __device__ __align__(256) int32_t g_dispatch_scratch[kNoAllocWords];

std::mutex g_scratch_mutex;
int32_t* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of g_dispatch_scratch on the current device.  In host code the array's name is
// only a handle for the runtime, not an address a kernel could use, so it is translated once
// per device with that device current.
cudaError_t scratch_address(int32_t** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        int32_t* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_dispatch_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

// One block: derives the bin layout from model_of_tenant and clears the words that must start
// at zero (the status word; the statistics are overwritten by the scan kernel).
__global__ void __launch_bounds__(256)
noalloc_setup_kernel(const int32_t* __restrict__ model_of_tenant, int n_tenants, int M, int E,
                     int32_t* __restrict__ tenant_local, int32_t* __restrict__ tenants_in_model,
                     int32_t* __restrict__ bin_base, int32_t* __restrict__ clean_model_of_tenant,
                     int32_t* __restrict__ stats, int32_t* __restrict__ status)
{
    const int tid = threadIdx.x;
    if (tid == 0) *status = 0;
    if (tid < 4) stats[tid] = 0;
    // thread m counts the tenants of model m in tenant order (sizes here are tiny)
    for (int m = tid; m < M; m += blockDim.x) {
        int n = 0;
        for (int u = 0; u < n_tenants; ++u) {
            int mu = model_of_tenant[u];
            if (mu < 0 || mu >= M) mu = 0;
            if (mu == m) { tenant_local[u] = n; clean_model_of_tenant[u] = mu; ++n; }
        }
        tenants_in_model[m] = n;
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int m = 0; m < M; ++m) { bin_base[m] = run; run += E * tenants_in_model[m]; }
        bin_base[M] = run;
    }
}

}  // namespace
}  // namespace faasmoe

extern "C" int moe_dispatch_noalloc(const int32_t* topk_idx, const int32_t* tenant_id, const int32_t* model_of_tenant,
                                    int T, int k, int E, int M, int n_tenants, int G, int32_t* perm, int32_t* inv_perm,
                                    int32_t* tenant_expert_count, int32_t* expert_off, int32_t* group_off,
                                    int32_t* status_out, void* stream)
{
    using namespace faasmoe;
    if (!topk_idx || !tenant_id || !model_of_tenant || !perm || !inv_perm || !expert_off) return MOE_ERR_NULL;
    if (T < 0 || k < 1 || k > kMaxTopK || E < 1 || E > kMaxExperts || k > E || M < 1 || M > kMaxExperts ||
        n_tenants < 1)
        return MOE_ERR_SHAPE;
    if (G < 1 || G > E) return MOE_ERR_G;
    if ((long long)T * k > (1 << 28) || (long long)E * n_tenants > kMaxBins) return MOE_ERR_SHAPE;
    const int R = T * k;
    const int nbins = E * n_tenants;
    const int nblk = (R + kDispatchChunk - 1) / kDispatchChunk;
    // scratch layout, in 32-bit words
    const long long o_stats = 0, o_status = 4, o_mot = 8, o_local = o_mot + n_tenants, o_tim = o_local + n_tenants,
                    o_base = o_tim + M, o_binoff = o_base + M + 1, o_blk = o_binoff + nbins + 1,
                    total = o_blk + (long long)nblk * nbins;
    if (total > kNoAllocWords) return MOE_ERR_UNSUPPORTED;     // beyond the fixed scratch: see the header
    if (T == 0) {
        // nothing to dispatch; the caller's status word is still cleared, as for any other call
        if (status_out && cudaMemsetAsync(status_out, 0, sizeof(int32_t), (cudaStream_t)stream) != cudaSuccess) return MOE_ERR_CUDA;
        return MOE_OK;
    }
    int32_t* s = nullptr;
    if (scratch_address(&s) != cudaSuccess) return MOE_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* status = status_out ? status_out : s + o_status;
    noalloc_setup_kernel<<<1, 256, 0, st>>>(model_of_tenant, n_tenants, M, E, s + o_local, s + o_tim, s + o_base,
                                            s + o_mot, s + o_stats, status);
    BinMap bm;
    bm.model_of_tenant = s + o_mot;
    bm.tenant_local = s + o_local;
    bm.bin_base = s + o_base;
    bm.tenants_in_model = s + o_tim;
    bm.n_tenants = n_tenants;
    bm.E = E;
    const size_t smem = (size_t)nbins * sizeof(int32_t);
    // stats[2] (cleared by the set-up kernel) counts the blocks that have finished
    dispatch_count_kernel<<<nblk, kCountThreads, smem, st>>>(topk_idx, tenant_id, nblk, nbins, R, k, E, M, G, n_tenants, bm,
                                                             s + o_blk, s + o_binoff, inv_perm, tenant_expert_count,
                                                             expert_off, group_off, s + o_stats, status, s + o_stats + 2, 0,
                                                             PlanArgs(), 0, nullptr, 0);
    dispatch_place_kernel<false><<<(R + 255) / 256, 256, 0, st>>>(R, k, nbins, s + o_blk, s + o_binoff, perm, inv_perm,
                                                                  nullptr, nullptr, 0, nullptr, 0, PlanArgs());
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
