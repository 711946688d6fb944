// CUDA-core expert execution: the plain, tile-wise SwiGLU FFN used for shapes the tensor-core
// path does not cover and as the A/B reference of that path.  (Paper Sec. 3: an expert block
// keeps no state and computes on the tokens it was sent; only activated experts are touched.)
#include <cuda_fp16.h>

#include "internal.h"

namespace faasmoe {

namespace {

constexpr int kRowsPerPass = 8;
constexpr int kColsPerBlock = 64;

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// weights bf16, activations fp16 (the shared expert's SwiGLU activations, see launch_experts_fma)
__device__ __forceinline__ void fma8_half(const uint4& w, const uint4& a, float& acc)
{
    const __nv_bfloat162* pw = reinterpret_cast<const __nv_bfloat162*>(&w);
    const __half2* pa = reinterpret_cast<const __half2*>(&a);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 fw = __bfloat1622float2(pw[i]);
        const float2 fa = __half22float2(pa[i]);
        acc = fmaf(fw.x, fa.x, acc);
        acc = fmaf(fw.y, fa.y, acc);
    }
}

__device__ __forceinline__ void fma8(const uint4& w, const uint4& a, float& acc)
{
    const __nv_bfloat162* pw = reinterpret_cast<const __nv_bfloat162*>(&w);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 fw = __bfloat1622float2(pw[i]);
        const float2 fa = __bfloat1622float2(pa[i]);
        acc = fmaf(fw.x, fa.x, acc);
        acc = fmaf(fw.y, fa.y, acc);
    }
}

// out[dst(r), c] = epi( W0[c,:] . act[r,:], W1[c,:] . act[r,:] ) for the rows r of one tile and
// 64 weight rows c.  SWIGLU: epi = silu(a) * b; otherwise epi = a (W1 unused).
// The shared expert's intermediate (SWIGLU && SHARED output, !SWIGLU && SHARED input) is fp16.
template <bool SWIGLU, bool SHARED>
__global__ void __launch_bounds__(256)
ffn_fma_kernel(const Tile* __restrict__ tiles, const int32_t* __restrict__ n_tiles_ptr, const bf16* __restrict__ act,
               int K, int ncols, PoolWeights pool, const ModelWeights* __restrict__ models, void* __restrict__ out_raw,
               int ld_out, const int32_t* __restrict__ dst_rows)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    bf16* a_s = reinterpret_cast<bf16*>(smem_raw);       // [kRowsPerPass][K]
    if ((int)blockIdx.x >= *n_tiles_ptr) return;
    const Tile tile = tiles[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kv = K >> 3;

    const bf16 *W0, *W1;
    if (SHARED) {
        const ModelWeights& mw = models[tile.slot];
        W0 = SWIGLU ? mw.ws_gate : mw.ws_down;
        W1 = SWIGLU ? mw.ws_up : nullptr;
    } else {
        const size_t per_slot = (size_t)ncols * K;
        W0 = (SWIGLU ? pool.w_gate : pool.w_down) + (size_t)tile.slot * per_slot;
        W1 = SWIGLU ? pool.w_up + (size_t)tile.slot * per_slot : nullptr;
    }

    for (int r0 = 0; r0 < tile.nrows; r0 += kRowsPerPass) {
        __syncthreads();
        for (int v = threadIdx.x; v < kRowsPerPass * kv; v += blockDim.x) {
            const int r = v / kv, kk = v - r * kv;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r0 + r < tile.nrows)
                val = reinterpret_cast<const uint4*>(act + (size_t)(tile.row0 + r0 + r) * K)[kk];
            reinterpret_cast<uint4*>(a_s)[v] = val;
        }
        __syncthreads();
        for (int cc = 0; cc < kColsPerBlock / 8; ++cc) {
            const int c = blockIdx.y * kColsPerBlock + warp * (kColsPerBlock / 8) + cc;
            if (c >= ncols) break;
            float acc0[kRowsPerPass], acc1[kRowsPerPass];
#pragma unroll
            for (int r = 0; r < kRowsPerPass; ++r) { acc0[r] = 0.f; acc1[r] = 0.f; }
            const uint4* w0 = reinterpret_cast<const uint4*>(W0 + (size_t)c * K);
            const uint4* w1 = SWIGLU ? reinterpret_cast<const uint4*>(W1 + (size_t)c * K) : nullptr;
            for (int v = lane; v < kv; v += 32) {
                const uint4 a = __ldg(w0 + v);
                uint4 b = make_uint4(0, 0, 0, 0);
                if (SWIGLU) b = __ldg(w1 + v);
#pragma unroll
                for (int r = 0; r < kRowsPerPass; ++r) {
                    const uint4 xv = reinterpret_cast<const uint4*>(a_s)[r * kv + v];
                    if (!SWIGLU && SHARED) fma8_half(a, xv, acc0[r]);
                    else fma8(a, xv, acc0[r]);
                    if (SWIGLU) fma8(b, xv, acc1[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < kRowsPerPass; ++r) {
                const float s0 = warp_sum_f(acc0[r]);
                const float s1 = SWIGLU ? warp_sum_f(acc1[r]) : 0.f;
                if (lane == r && r0 + r < tile.nrows) {
                    const float val = SWIGLU ? (s0 / (1.f + expf(-s0))) * s1 : s0;
                    const int row = tile.row0 + r0 + r;
                    const int drow = dst_rows ? dst_rows[row] : row;
                    const size_t o = (size_t)drow * ld_out + c;
                    if (!SWIGLU) reinterpret_cast<float*>(out_raw)[o] = val;                       // y: fp32
                    else if (SHARED) reinterpret_cast<__half*>(out_raw)[o] = __float2half_rn(fminf(fmaxf(val, -65504.f), 65504.f));  // hs: fp16
                    else reinterpret_cast<bf16*>(out_raw)[o] = __float2bfloat16_rn(val);            // h: bf16
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_experts_fma(moe_ctx* c, int layer, const bf16* x_or_xs, const bf16* x_perm, int T, float* y_perm,
                               float* y_shared, const int32_t* shared_dst_rows, cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const PoolWeights pool = c->pools[layer];
    const ModelWeights* models = c->d_models + (size_t)layer * g.n_models;
    const int H = g.hidden, I = g.inter, Is = g.shared_inter;
    const int* n_tiles = c->ws.plan_counts;

    auto set_smem = [](const void* fn, size_t bytes) {
        cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    };
    const bool shared = y_shared && Is > 0;
    const size_t smem_h = (size_t)kRowsPerPass * H * sizeof(bf16);
    const size_t smem_i = (size_t)kRowsPerPass * I * sizeof(bf16);
    const size_t smem_is = (size_t)kRowsPerPass * Is * sizeof(bf16);
    set_smem((const void*)ffn_fma_kernel<true, false>, smem_h);
    set_smem((const void*)ffn_fma_kernel<false, false>, smem_i);
    if (shared) {
        set_smem((const void*)ffn_fma_kernel<true, true>, smem_h);
        set_smem((const void*)ffn_fma_kernel<false, true>, smem_is);
    }
    // gate/up + SwiGLU
    dim3 g1(c->max_tiles, (I + kColsPerBlock - 1) / kColsPerBlock);
    ffn_fma_kernel<true, false><<<g1, 256, smem_h, st>>>(c->ws.tiles, n_tiles, x_perm, H, I, pool, nullptr, c->ws.h, I,
                                                         nullptr);
    if (shared) {
        dim3 gs1(c->max_stiles, (Is + kColsPerBlock - 1) / kColsPerBlock);
        ffn_fma_kernel<true, true><<<gs1, 256, smem_h, st>>>(c->ws.stiles, n_tiles + 1, x_or_xs, H, Is, pool, models,
                                                             c->ws.hs, Is, nullptr);
    }
    stage_mark(c, st, kEvGateUp);
    // down projection
    dim3 g2(c->max_tiles, (H + kColsPerBlock - 1) / kColsPerBlock);
    ffn_fma_kernel<false, false><<<g2, 256, smem_i, st>>>(c->ws.tiles, n_tiles, c->ws.h, I, H, pool, nullptr, y_perm, H,
                                                          nullptr);
    if (shared) {
        dim3 gs2(c->max_stiles, (H + kColsPerBlock - 1) / kColsPerBlock);
        ffn_fma_kernel<false, true><<<gs2, 256, smem_is, st>>>(c->ws.stiles, n_tiles + 1, (const bf16*)c->ws.hs, Is, H, pool, models,
                                                               y_shared, H, shared_dst_rows);
    }
    stage_mark(c, st, kEvDown);
    c->launches += shared ? 4 : 2;
    return cudaGetLastError();
}

}  // namespace faasmoe
