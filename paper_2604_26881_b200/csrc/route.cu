// Gating network: router logits, fp32 softmax, top-k by warp shuffles, shared-expert gate.
// (Paper Sec. 2.1: the gating network selects the top-k experts of each token; Sec. 3: it
// runs in the orchestrator, ahead of the expert blocks.)
#include "internal.h"

namespace faasmoe {

namespace {

constexpr int kRouteWarps = 8;
constexpr int kExpertsPerStage = 8;    // router rows staged in shared memory at a time
constexpr int kMaxChunks = kMaxExperts / 32;

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc)
{
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 fa = __bfloat1622float2(pa[i]);
        float2 fb = __bfloat1622float2(pb[i]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
    }
    return acc;
}

// One warp owns TPW tokens.  The block stages kExpertsPerStage router rows of one model in
// shared memory; every warp whose tokens use that model consumes them.  Tokens of a block
// may belong to different models, so the block walks the models its tokens use.
template <int TPW>
__global__ void __launch_bounds__(kRouteWarps * 32)
route_kernel(const bf16* __restrict__ x, const int32_t* __restrict__ tenant_id, int T, int H, int E, int k,
             int n_tenants, int n_models, const int32_t* __restrict__ model_of_tenant,
             const ModelWeights* __restrict__ models, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
             float* __restrict__ shared_gate, uint8_t* __restrict__ tie_flag, int32_t* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    bf16* w_s = reinterpret_cast<bf16*>(smem_raw);                       // [kExpertsPerStage][H]
    bf16* x_s = w_s + (size_t)kExpertsPerStage * H;                      // [warps*TPW][H]
    __shared__ int s_model_used[kRouteWarps * TPW];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tok0 = (blockIdx.x * kRouteWarps + warp) * TPW;
    const int nchunks = (E + 31) >> 5;
    const int hv = H >> 3;   // 16-byte vectors per row

    int model[TPW];
    bool valid[TPW], bad[TPW];
    float z[TPW][kMaxChunks];
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
        const int t = tok0 + i;
        valid[i] = t < T;
        bad[i] = false;
        model[i] = -1;
        if (valid[i]) {
            int u = tenant_id[t];
            if (u < 0 || u >= n_tenants) { bad[i] = true; u = 0; }
            model[i] = model_of_tenant[u];
            const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * H);
            uint4* dst = reinterpret_cast<uint4*>(x_s + (size_t)(warp * TPW + i) * H);
            for (int v = lane; v < hv; v += 32) dst[v] = src[v];
        }
        if (lane == 0) s_model_used[warp * TPW + i] = model[i];
#pragma unroll
        for (int c = 0; c < kMaxChunks; ++c) z[i][c] = -INFINITY;
    }
    __syncthreads();

    for (int m = 0; m < n_models; ++m) {
        bool used = false;
        for (int i = 0; i < kRouteWarps * TPW; ++i) used |= (s_model_used[i] == m);
        if (!used) continue;                         // uniform across the block
        const bf16* rw = models[m].router_w;
        const float* rb = models[m].router_bias;
        for (int e0 = 0; e0 < E; e0 += kExpertsPerStage) {
            const int ne = min(kExpertsPerStage, E - e0);
            __syncthreads();
            {
                const uint4* src = reinterpret_cast<const uint4*>(rw + (size_t)e0 * H);
                uint4* dst = reinterpret_cast<uint4*>(w_s);
                for (int v = threadIdx.x; v < ne * hv; v += blockDim.x) dst[v] = src[v];
            }
            __syncthreads();
#pragma unroll
            for (int i = 0; i < TPW; ++i) {
                if (model[i] != m) continue;        // uniform within the warp
                const uint4* xv = reinterpret_cast<const uint4*>(x_s + (size_t)(warp * TPW + i) * H);
                for (int ee = 0; ee < ne; ++ee) {
                    const uint4* wv = reinterpret_cast<const uint4*>(w_s + (size_t)ee * H);
                    float acc = 0.f;
                    for (int v = lane; v < hv; v += 32) acc = dot8(xv[v], wv[v], acc);
                    acc = warp_sum(acc);
                    const int e = e0 + ee;
                    if (rb) acc += rb[e];
                    if ((e & 31) == lane) {
#pragma unroll
                        for (int c = 0; c < kMaxChunks; ++c) if (c == (e >> 5)) z[i][c] = acc;
                    }
                }
            }
        }
    }

#pragma unroll
    for (int i = 0; i < TPW; ++i) {
        if (!valid[i]) continue;
        const int t = tok0 + i;
        // softmax over the E logits held as z[i][c] on lane (e & 31)
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < kMaxChunks; ++c) if (c < nchunks) zmax = fmaxf(zmax, z[i][c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
        float p[kMaxChunks];
        float den = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxChunks; ++c) {
            const bool live = c < nchunks && (c * 32 + lane) < E;
            p[c] = live ? expf(z[i][c] - zmax) : 0.f;
            den += p[c];
        }
        den = warp_sum(den);
#pragma unroll
        for (int c = 0; c < kMaxChunks; ++c) p[c] = ((c * 32 + lane) < E && c < nchunks) ? p[c] / den : -1.f;

        // k (+1) rounds of warp arg-max; ties go to the lower expert id
        const int rounds = (k < E) ? k + 1 : k;
        float prev = 0.f;
        uint8_t flag = 0;
        for (int j = 0; j < rounds; ++j) {
            float bv = -1.f;
            int bi = 0x7fffffff;
#pragma unroll
            for (int c = 0; c < kMaxChunks; ++c) {
                if (c < nchunks && p[c] > bv) { bv = p[c]; bi = c * 32 + lane; }   // ascending c: lower id wins ties
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (j > 0 && (prev - bv) < 1e-5f * prev) flag = 1;
            prev = bv;
            if (j < k && lane == 0) {
                topk_idx[(size_t)t * k + j] = bad[i] ? j : bi;
                topk_w[(size_t)t * k + j] = bad[i] ? 0.f : bv;
            }
            if ((bi & 31) == lane) {
#pragma unroll
                for (int c = 0; c < kMaxChunks; ++c) if (c == (bi >> 5)) p[c] = -1.f;   // taken
            }
        }
        if (tie_flag && lane == 0) tie_flag[t] = flag;
        if (shared_gate) {
            float g = 0.f;
            const bf16* sg = models[model[i]].shared_gate_w;
            if (sg && !bad[i]) {
                const uint4* xv = reinterpret_cast<const uint4*>(x_s + (size_t)(warp * TPW + i) * H);
                const uint4* wv = reinterpret_cast<const uint4*>(sg);
                float acc = 0.f;
                for (int v = lane; v < hv; v += 32) acc = dot8(xv[v], __ldg(wv + v), acc);
                acc = warp_sum(acc);
                g = 1.f / (1.f + expf(-acc));
            } else if (!bad[i]) {
                g = 0.5f;
            }
            if (lane == 0) shared_gate[t] = g;
        }
        if (bad[i] && lane == 0) atomicOr(status, MOE_DEV_BAD_TENANT);
    }
}

}  // namespace

cudaError_t launch_route(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                         float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st)
{
    const bool tc = c->route_path != MOE_PATH_FMA && route_tc_supported(c);      // (x is 16-byte aligned: checked at the ABI)
    return tc ? launch_route_tc(c, layer, x, tenant_id, T, topk_idx, topk_w, shared_gate, tie_flag, st)
              : launch_route_fma(c, layer, x, tenant_id, T, topk_idx, topk_w, shared_gate, tie_flag, st);
}

cudaError_t launch_route_fma(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                             float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const ModelWeights* models = c->d_models + (size_t)layer * g.n_models;
    // small batches: one token per warp so that the tokens spread over many SMs
    const size_t smem4 = (size_t)(kExpertsPerStage + kRouteWarps * 4) * g.hidden * sizeof(bf16);
    const bool small = T <= 1024 || smem4 > 200 * 1024;
    const int tpw = small ? 1 : 4;
    const int tok_per_block = kRouteWarps * tpw;
    const int blocks = (T + tok_per_block - 1) / tok_per_block;
    const size_t smem = (size_t)(kExpertsPerStage + tok_per_block) * g.hidden * sizeof(bf16);
    if (small) {
        cudaFuncSetAttribute(route_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        route_kernel<1><<<blocks, kRouteWarps * 32, smem, st>>>(x, tenant_id, T, g.hidden, g.n_experts, g.top_k,
            g.n_tenants, g.n_models, c->d_model_of_tenant, models, topk_idx, topk_w, shared_gate, tie_flag, c->ws.status);
    } else {
        cudaFuncSetAttribute(route_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        route_kernel<4><<<blocks, kRouteWarps * 32, smem, st>>>(x, tenant_id, T, g.hidden, g.n_experts, g.top_k,
            g.n_tenants, g.n_models, c->d_model_of_tenant, models, topk_idx, topk_w, shared_gate, tie_flag, c->ws.status);
    }
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
