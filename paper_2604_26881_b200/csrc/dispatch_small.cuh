// The one-block dispatch of small batches as a device function: the kernel of its own (dispatch.cu) and the
// router kernel of a one-tile batch (route_tc.cu), which runs it behind its top-k step, share it.
#pragma once

#include "internal.h"
#include "plan.cuh"
#include "scan.cuh"

namespace faasmoe {

// bin of a routed row: bins are laid out (model, expert, tenant-of-that-model)
struct BinMap {
    const int32_t* model_of_tenant;
    const int32_t* tenant_local;
    const int32_t* bin_base;          // [M+1]
    const int32_t* tenants_in_model;  // [M]
    int n_tenants, E;
};

__device__ __forceinline__ int row_bin(const BinMap& bm, int tenant, int expert, int32_t* status)
{
    if (tenant < 0 || tenant >= bm.n_tenants) { atomicOr(status, MOE_DEV_BAD_TENANT); tenant = 0; }
    if (expert < 0 || expert >= bm.E) { atomicOr(status, MOE_DEV_BAD_EXPERT); expert = 0; }
    const int m = bm.model_of_tenant[tenant];
    return bm.bin_base[m] + expert * bm.tenants_in_model[m] + bm.tenant_local[tenant];
}

// Block-wide: exclusive scan of the per-bin totals in s_tot (in key order), then the offset tables
// the caller sees and the invocation statistics.  s_tot holds the offsets afterwards.
static __device__ void scan_and_tables(int32_t* s_tot, int32_t* s_part /* [33] */, int32_t* s_count /* [2] */,
                                int nbins, int R, int E, int M, int G, int n_tenants, const BinMap& bm,
                                int32_t* __restrict__ bin_off /* may be null */,
                                int32_t* __restrict__ tenant_expert_count, int32_t* __restrict__ expert_off,
                                int32_t* __restrict__ group_off, int32_t* __restrict__ stats, int private_mode,
                                const int32_t* __restrict__ block_table = nullptr, int table_blocks = 0)
{
    const int tid = threadIdx.x, nth = blockDim.x;
    if (tid < 2) s_count[tid] = 0;
    if (tenant_expert_count) {
        for (int i = tid; i < n_tenants * E; i += nth) {
            const int u = i / E, e = i - u * E;
            const int m = bm.model_of_tenant[u];
            tenant_expert_count[i] = s_tot[bm.bin_base[m] + e * bm.tenants_in_model[m] + bm.tenant_local[u]];
        }
    }
    __syncthreads();
    block_scan_exclusive(s_tot, nbins, s_part);
    if (bin_off) {
        for (int b = tid; b < nbins; b += nth) bin_off[b] = s_tot[b];
        if (tid == 0) bin_off[nbins] = R;
    }
    // expert_off[m*E + e] = offset of the first bin of (m, e); a model without tenants owns
    // no bins, so its experts start where the next model's bins start
    for (int i = tid; i <= M * E; i += nth) {
        int v = R;
        if (i < M * E) {
            const int m = i / E, e = i - m * E;
            const int first = bm.bin_base[m] + e * bm.tenants_in_model[m];
            v = (first < nbins) ? s_tot[first] : R;
        }
        expert_off[i] = v;
    }
    __syncthreads();
    if (block_table) {
        // Blocks given by a table (load-aware formation, Sec. 5) are sets of experts, not ranges of rows: group_off
        // then holds the running sum of the rows every block receives, in block order.  Sizes are small (M * B blocks,
        // E experts each): plain loops.
        const int B = table_blocks;
        for (int i = tid; i < M * B; i += nth) {
            const int m = i / B, b = i - m * B;
            int rows = 0;
            for (int e = 0; e < E; ++e)
                if (block_table[m * E + e] == b) rows += expert_off[m * E + e + 1] - expert_off[m * E + e];
            if (rows > 0 && !private_mode) atomicAdd(&s_count[0], 1);
            if (group_off) group_off[i + 1] = rows;
        }
        __syncthreads();
        if (tid == 0 && group_off) {
            int run = 0;
            group_off[0] = 0;
            for (int i = 1; i <= M * B; ++i) { run += group_off[i]; group_off[i] = run; }
        }
        if (private_mode) {
            for (int i = tid; i < n_tenants * B; i += nth) {
                const int u = i / B, b = i - u * B;
                const int m = bm.model_of_tenant[u];
                const int tim = bm.tenants_in_model[m], ul = bm.tenant_local[u];
                bool any = false;
                for (int e = 0; e < E; ++e) {
                    if (block_table[m * E + e] != b) continue;
                    const int bin = bm.bin_base[m] + e * tim + ul;
                    const int end = bin + 1 < nbins ? s_tot[bin + 1] : R;
                    any = any || end > s_tot[bin];
                }
                if (any) atomicAdd(&s_count[0], 1);
            }
        }
        for (int i = tid; i < M * E; i += nth)
            if (expert_off[i + 1] > expert_off[i]) atomicAdd(&s_count[1], 1);
        __syncthreads();
        if (tid < 2) stats[tid] = s_count[tid];
        return;
    }
    // expert blocks of G experts; invocation statistics
    const int B = (E + G - 1) / G;
    for (int i = tid; i <= M * B; i += nth) {
        int v = R;
        if (i < M * B) {
            const int m = i / B, b = i - m * B;
            const int e0 = b * G, e1 = min(E, e0 + G);
            v = expert_off[m * E + e0];
            if (!private_mode && expert_off[m * E + e1] > v) atomicAdd(&s_count[0], 1);
        }
        if (group_off) group_off[i] = v;
    }
    if (private_mode) {
        // private orchestrators (Sec. 4.2): every tenant batches its own tokens, so an invocation is a pair
        // (tenant, block of its model) with at least one row
        for (int i = tid; i < n_tenants * B; i += nth) {
            const int u = i / B, b = i - u * B;
            const int m = bm.model_of_tenant[u];
            const int tim = bm.tenants_in_model[m], ul = bm.tenant_local[u];
            bool any = false;
            for (int e = b * G; e < min(E, (b + 1) * G); ++e) {
                const int bin = bm.bin_base[m] + e * tim + ul;
                const int end = bin + 1 < nbins ? s_tot[bin + 1] : R;
                any = any || end > s_tot[bin];
            }
            if (any) atomicAdd(&s_count[0], 1);
        }
    }
    for (int i = tid; i < M * E; i += nth)
        if (expert_off[i + 1] > expert_off[i]) atomicAdd(&s_count[1], 1);
    __syncthreads();
    if (tid < 2) stats[tid] = s_count[tid];
}

// Arguments of the one-block dispatch (one kernel parameter).
struct SmallDispatchArgs {
    int enabled;                      // (router kernel: 0 = no dispatch behind the top-k step)
    const int32_t* topk_idx;
    const int32_t* tenant_id;
    int R, k;
    BinMap bm;
    int nbins, E, M, G, n_tenants;
    int32_t* perm;
    int32_t* inv_perm;
    int32_t* tenant_expert_count;
    int32_t* expert_off;
    int32_t* group_off;
    int32_t* stats;
    int32_t* status;
    const bf16* x;
    bf16* x_perm;                     // null: no gather
    int H;
    int do_plan, plan_ints;
    PlanArgs pa;
    int32_t* bin_off;                 // null unless the orchestrators are private
    int private_mode;
    const int32_t* block_table;
    int table_blocks;
};

// Whole block, any block size that is a multiple of 32.  s_tot: [nbins] ints, then the plan's scratch (plan_ints),
// then one unsigned short per row.  Histogram, scan, tables, stable ranks (one warp walks the rows in order), the
// expert work plan and the gather of the rows.  Same results as the multi-block kernels.  The expert ids are read
// past the L1 (the calling kernel may have written them itself).
__device__ __forceinline__ void dispatch_small_body(const SmallDispatchArgs& a, int32_t* s_tot)
{
    __shared__ int32_t s_part[33];
    __shared__ int32_t s_count[2];
    const int tid = threadIdx.x, nth = blockDim.x;
    const int R = a.R, k = a.k, nbins = a.nbins;
    int32_t* __restrict__ perm = a.perm;
    int32_t* __restrict__ inv_perm = a.inv_perm;
    unsigned short* s_bin = reinterpret_cast<unsigned short*>(s_tot + nbins + a.plan_ints);
    for (int b = tid; b < nbins; b += nth) s_tot[b] = 0;
    __syncthreads();
    for (int r = tid; r < R; r += nth) {
        const int bin = row_bin(a.bm, a.tenant_id[r / k], __ldcg(a.topk_idx + r), a.status);
        s_bin[r] = (unsigned short)bin;      // nbins <= 8192: fits; the ranking pass below reads it back
        atomicAdd(&s_tot[bin], 1);
    }
    __syncthreads();
    scan_and_tables(s_tot, s_part, s_count, nbins, R, a.E, a.M, a.G, a.n_tenants, a.bm, a.bin_off, a.tenant_expert_count,
                    a.expert_off, a.group_off, a.stats, a.private_mode, a.block_table, a.table_blocks);
    __syncthreads();
    if (tid < 32) {                           // s_tot now holds the next free position of every bin
        const int lane = tid;
        for (int rr = 0; rr < R; rr += 32) {
            const int r = rr + lane;
            const bool live = r < R;
            int bin = -1 - lane;
            if (live) bin = s_bin[r];
            const unsigned peers = __match_any_sync(0xffffffffu, bin);
            const int leader = __ffs(peers) - 1;
            const int rank = __popc(peers & ((1u << lane) - 1u));
            int start = 0;
            if (live && lane == leader) { start = s_tot[bin]; s_tot[bin] = start + __popc(peers); }
            start = __shfl_sync(0xffffffffu, start, leader);
            if (live) { perm[start + rank] = r; inv_perm[r] = start + rank; }
            __syncwarp();
        }
    }
    if (a.do_plan) {
        __syncthreads();                      // expert_off (written above) is visible to the block
        plan_body(a.expert_off, a.pa, s_tot + nbins, s_part);
    }
    if (a.x_perm) {
        __syncthreads();                      // perm is complete and visible to the block
        const int warp = tid >> 5, lane = tid & 31, nw = nth >> 5;
        for (int pos = warp; pos < R; pos += nw) {
            const int t = perm[pos] / k;
            const uint4* src = reinterpret_cast<const uint4*>(a.x + (size_t)t * a.H);
            uint4* dst = reinterpret_cast<uint4*>(a.x_perm + (size_t)pos * a.H);
            for (int v = lane; v < (a.H >> 3); v += 32) dst[v] = src[v];
        }
    }
}

}  // namespace faasmoe
