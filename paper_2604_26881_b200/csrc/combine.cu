// Aggregation of expert outputs per token (paper Sec. 3: the orchestrator aggregates the
// results of the expert functions; Sec. 4.2 lists it among the orchestrator's duties), and the RMSNorm / residual
// add of the stacked-block configuration.
#include "internal.h"

namespace faasmoe {

namespace {

__device__ __forceinline__ void unpack8(const uint4& v, float* f)
{
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __bfloat1622float2(p[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

__device__ __forceinline__ void load8(const float* p, float* f)
{
    const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
    f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

__device__ __forceinline__ uint4 pack8(const float* f)
{
    uint4 v;
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
}

// out[t] = residual[t] + sum_j w[t,j] * y_perm[inv_perm[t*k+j]] + s[t] * y_shared[t]
// (fp32, fixed order: residual, j = 0..k-1, shared), one rounding to bf16.
// One thread per 8 consecutive features.
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ y_perm, const int32_t* __restrict__ inv_perm, const float* __restrict__ topk_w,
               const float* __restrict__ y_shared, const float* __restrict__ shared_gate,
               const bf16* residual, int T, int H, int k, bf16* out)
{
    pdl_wait();
    pdl_launch_dependents();
    const int hv = H >> 3;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= (long long)T * hv) return;
    const int t = (int)(gid / hv), v = (int)(gid - (long long)t * hv);
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    // All loads are issued before the first sum: positions and weights of the k rows, then the rows themselves (four
    // at a time), the shared row and the residual.  With few tokens this kernel is a chain of memory latencies, and
    // position -> row, once per j, made it k times as long.  The order of the sums stays residual, j = 0..k-1, shared.
    int rj[kMaxTopK];
    float wj[kMaxTopK];
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) {
        rj[j] = j < k ? inv_perm[(size_t)t * k + j] : 0;
        wj[j] = j < k ? topk_w[(size_t)t * k + j] : 0.f;
    }
    float sh[8];
    float s = 0.f;
    if (y_shared) {
        s = shared_gate[t];
        load8(y_shared + (size_t)t * H + 8 * v, sh);
    }
    if (residual) unpack8(reinterpret_cast<const uint4*>(residual + (size_t)t * H)[v], acc);
#pragma unroll
    for (int j0 = 0; j0 < kMaxTopK; j0 += 4) {
        if (j0 < k) {
            float rows[4][8];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
                if (j0 + jj < k) load8(y_perm + (size_t)rj[j0 + jj] * H + 8 * v, rows[jj]);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                if (j0 + jj < k) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = fmaf(wj[j0 + jj], rows[jj][i], acc[i]);
                }
            }
        }
    }
    if (y_shared) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = fmaf(s, sh[i], acc[i]);
    }
    reinterpret_cast<uint4*>(out + (size_t)t * H)[v] = pack8(acc);
}

// xn[t] = bf16( x[t] * rsqrt(mean(x[t]^2) + eps) * g ), fp32 arithmetic.  One warp per token.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const bf16* __restrict__ x, const int32_t* __restrict__ tenant_id, int T, int H, float eps,
               int n_tenants, const int32_t* __restrict__ model_of_tenant, const ModelWeights* __restrict__ models,
               bf16* __restrict__ xn)
{
    pdl_wait();
    pdl_launch_dependents();
    const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (t >= T) return;
    int u = tenant_id[t];
    if (u < 0 || u >= n_tenants) u = 0;
    const bf16* g = models[model_of_tenant[u]].rms_w;
    const uint4* xv = reinterpret_cast<const uint4*>(x + (size_t)t * H);
    const uint4* gv = reinterpret_cast<const uint4*>(g);
    const int hv = H >> 3;
    float ss = 0.f, f[8], w[8];
    for (int v = lane; v < hv; v += 32) {
        unpack8(xv[v], f);
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float r = rsqrtf(ss / (float)H + eps);
    for (int v = lane; v < hv; v += 32) {
        unpack8(xv[v], f);
        unpack8(__ldg(gv + v), w);
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = f[i] * r * w[i];
        reinterpret_cast<uint4*>(xn + (size_t)t * H)[v] = pack8(f);
    }
}

}  // namespace

cudaError_t launch_combine(moe_ctx* c, const float* y_perm, const int32_t* inv_perm, const float* topk_w,
                           const float* y_shared, const float* shared_gate, const bf16* residual, int T, bf16* out,
                           cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const long long n = (long long)T * (g.hidden >> 3);
    const int blocks = (int)((n + 255) / 256);
    launch_pdl(combine_kernel, dim3(blocks), dim3(256), 0, st, y_perm, inv_perm, topk_w, y_shared, shared_gate, residual, T, g.hidden,
                                           g.top_k, out);
    c->launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, bf16* xn,
                           cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const int blocks = (T * 32 + 255) / 256;
    launch_pdl(rmsnorm_kernel, dim3(blocks), dim3(256), 0, st, x, tenant_id, T, g.hidden, g.rms_eps, g.n_tenants, c->d_model_of_tenant,
                                           c->d_models + (size_t)layer * g.n_models, xn);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
