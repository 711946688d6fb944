// Tensor-core expert execution for sm_100a: one persistent, warp-specialised grouped GEMM
// (TMA -> shared memory -> tcgen05.mma -> TMEM -> registers) used twice per layer:
//   gate/up:  h[r, c]  = silu(W_g[c,:] . x[r,:]) * (W_u[c,:] . x[r,:])        (SwiGLU in the epilogue)
//   down:     y[r, c]  = W_d[c,:] . h[r,:]
// (paper Sec. 3: an expert block computes on the tokens assigned to it; only activated experts are
// touched.)  The weight rows are the M operand of the MMA (128 rows per instruction, two
// instructions per unit), the tokens of one expert tile are the N operand (16..128, a multiple of
// 16), so a decode-sized tile streams each weight byte once through a narrow MMA and a prefill tile
// uses the full 128x128 shape with no padding of ragged expert segments beyond 16 rows.
// Routed-expert units and shared-expert units ride in the same launch.
#include <cuda_fp16.h>

#include <cstdio>
#include <cstring>

#include "internal.h"
#include "tc_ptx.cuh"

namespace faasmoe {

namespace {

using namespace tc;

constexpr int kStages = 4;
constexpr int kBK = 64;                       // K elements per stage = one 128-byte swizzle row
constexpr int kABytes = 128 * kBK * 2;        // one 128-row weight tile: 16 KB
constexpr int kBBytes = kTileRows * kBK * 2;  // up to 128 token rows: 16 KB
constexpr int kStageBytes = 2 * kABytes + kBBytes;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kThreads = 192;                 // warp 0: TMA, warp 1: MMA + TMEM, warps 2-5: epilogue
constexpr uint32_t kTmemCols = 512;           // 2 buffers x (2 accumulators x 128 columns)

struct GemmParams {
    const Unit* units;
    const int32_t* n_units;
    const Tile* tiles;
    const Tile* stiles;
    const CUtensorMap* amaps;     // [0],[1]: routed A0/A1; [2+2m],[3+2m]: shared A0/A1 of model m
    int k_routed, k_shared;       // contraction lengths
    int rows_per_slot;            // weight rows per pool slot in the routed A maps
    int cb_stride, a1_off;        // A0 row = base + cb*cb_stride, A1 row = A0 row + a1_off
    void* out_routed;
    void* out_shared;
    int ld_routed, ld_shared;
    const int32_t* shared_dst_rows;
    uint32_t idesc_fmt_routed, idesc_fmt_shared;   // operand format bits of the instruction descriptor
    int stream_weights;           // 1: every weight tile is read once (small batch): mark it evict-first in L2
    int32_t* status;
};

struct UnitInfo {
    int a0_row, a1_row, amap0, amap1;
    int b_row0, nrows, npad, ksteps, shared, cb;
};

__device__ __forceinline__ UnitInfo decode_unit(const GemmParams& p, int u)
{
    const Unit un = p.units[u];
    UnitInfo ui;
    ui.shared = un.tile < 0;
    const Tile t = ui.shared ? p.stiles[~un.tile] : p.tiles[un.tile];
    ui.cb = un.colblock;
    const int base = ui.shared ? 0 : t.slot * p.rows_per_slot;
    ui.a0_row = base + un.colblock * p.cb_stride;
    ui.a1_row = ui.a0_row + p.a1_off;
    ui.amap0 = ui.shared ? 2 + 2 * t.slot : 0;
    ui.amap1 = ui.amap0 + 1;
    ui.b_row0 = t.row0;
    ui.nrows = t.nrows;
    ui.npad = (t.nrows + 15) & ~15;
    ui.ksteps = (ui.shared ? p.k_shared : p.k_routed) / kBK;
    return ui;
}

// MODE 0: gate/up + SwiGLU (output bf16 for routed units, fp16 for shared units)
// MODE 1: down projection (output fp32)
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_kernel(const GemmParams p, const __grid_constant__ CUtensorMap b_routed128,
                    const __grid_constant__ CUtensorMap b_routed16, const __grid_constant__ CUtensorMap b_shared128,
                    const __grid_constant__ CUtensorMap b_shared16)
{
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
    const uint32_t bars = smem_base + kStages * kStageBytes;                   // 8-byte barriers after the tiles
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kStages;
    const uint32_t bar_tfull = bars + 16 * kStages, bar_tempty = bar_tfull + 16;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_units = *p.n_units;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer (one lane) ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t armed = 0, armed_phase = 0;     // bit s: stage s has a load in flight / its phase
            bool ok = true;
            const uint64_t pol_w = p.stream_weights ? l2_evict_first() : l2_evict_last();
            const uint64_t pol_x = l2_evict_last();
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
                const UnitInfo ui = decode_unit(p, u);
                const CUtensorMap* ma0 = p.amaps + ui.amap0;
                const CUtensorMap* ma1 = p.amaps + ui.amap1;
                const CUtensorMap* mb128 = ui.shared ? &b_shared128 : &b_routed128;
                const CUtensorMap* mb16 = ui.shared ? &b_shared16 : &b_routed16;
                for (int ks = 0; ks < ui.ksteps; ++ks) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, &s_abort, p.status)) { ok = false; break; }
                    const uint32_t sa0 = smem_base + stage * kStageBytes, sa1 = sa0 + kABytes, sb = sa1 + kABytes;
                    const uint32_t full = bar_full + 8 * stage;
                    mbar_expect_tx(full, 2 * kABytes + ui.npad * kBK * 2);
                    armed |= 1u << stage;
                    armed_phase = (armed_phase & ~(1u << stage)) | (phase << stage);
                    tma_load_2d_hint(sa0, ma0, full, ks * kBK, ui.a0_row, pol_w);
                    tma_load_2d_hint(sa1, ma1, full, ks * kBK, ui.a1_row, pol_w);
                    if (ui.npad == kTileRows) {
                        tma_load_2d_hint(sb, mb128, full, ks * kBK, ui.b_row0, pol_x);
                    } else {
                        for (int j = 0; j < ui.npad; j += 16)
                            tma_load_2d_hint(sb + j * kBK * 2, mb16, full, ks * kBK, ui.b_row0 + j, pol_x);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                // gave up: let the copies already in flight land before the block exits
                for (int s = 0; s < kStages; ++s)
                    if (armed & (1u << s)) mbar_wait(bar_full + 8 * s, (armed_phase >> s) & 1u, &s_abort, p.status);
            }
        }
        __syncwarp();      // the whole warp reaches the block barrier below together
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane) ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
                const UnitInfo ui = decode_unit(p, u);
                const uint32_t fmt = ui.shared ? p.idesc_fmt_shared : p.idesc_fmt_routed;
                const uint32_t idesc = (1u << 4) | fmt | ((uint32_t)(ui.npad >> 3) << 17) | ((128u >> 4) << 24);
                if (!mbar_wait(bar_tempty + 8 * buf, bphase ^ 1, &s_abort, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + buf * 256, d1 = d0 + 128;
                for (int ks = 0; ks < ui.ksteps; ++ks) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, &s_abort, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa0 = smem_base + stage * kStageBytes, sa1 = sa0 + kABytes, sb = sa1 + kABytes;
                    const uint64_t da0 = smem_desc_sw128(sa0), da1 = smem_desc_sw128(sa1), db = smem_desc_sw128(sb);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        const uint32_t acc = (ks | kk) ? 1u : 0u;
                        const uint64_t adv = (uint64_t)(kk * 32 >> 4);      // 16 elements = 32 bytes along K
                        umma_bf16(d0, da0 + adv, db + adv, idesc, acc);
                        umma_bf16(d1, da1 + adv, db + adv, idesc, acc);
                    }
                    umma_commit(bar_empty + 8 * stage);      // frees the stage when these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit(bar_tfull + 8 * buf);            // accumulators complete
                if (++buf == 2) { buf = 0; bphase ^= 1; }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: 4 warps, one TMEM lane quarter each ----------------
        const int quarter = warp & 3;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int row_in_block = quarter * 32 + lane;       // weight row inside the 128-row tile
        uint32_t buf = 0, bphase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
            const UnitInfo ui = decode_unit(p, u);
            // one decision for the whole warp: the TMEM loads below are warp-wide instructions
            ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * buf, bphase, &s_abort, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d0 = tmem_base + lane_addr + buf * 256, d1 = d0 + 128;
            const int ld = ui.shared ? p.ld_shared : p.ld_routed;
            for (int c0 = 0; c0 < ui.npad; c0 += 16) {
                uint32_t r0[16], r1[16];
                tmem_ld16(d0 + c0, r0);
                tmem_ld16(d1 + c0, r1);
                tmem_ld_wait();
                if (MODE == 0) {
                    const int col = ui.cb * 128 + row_in_block;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = c0 + j;
                        if (n < ui.nrows) {
                            const float g = __uint_as_float(r0[j]), up = __uint_as_float(r1[j]);
                            const float v = (g / (1.f + __expf(-g))) * up;
                            const size_t o = (size_t)(ui.b_row0 + n) * ld + col;
                            if (ui.shared) reinterpret_cast<__half*>(p.out_shared)[o] = __float2half_rn(v);
                            else reinterpret_cast<bf16*>(p.out_routed)[o] = __float2bfloat16_rn(v);
                        }
                    }
                } else {
                    const int col = ui.cb * 256 + row_in_block;
                    float* out = reinterpret_cast<float*>(ui.shared ? p.out_shared : p.out_routed);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = c0 + j;
                        if (n < ui.nrows) {
                            int row = ui.b_row0 + n;
                            if (ui.shared && p.shared_dst_rows) row = p.shared_dst_rows[row];
                            out[(size_t)row * ld + col] = __uint_as_float(r0[j]);
                            out[(size_t)row * ld + col + 128] = __uint_as_float(r1[j]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
            if (++buf == 2) { buf = 0; bphase ^= 1; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

__global__ void bf16_to_fp16_kernel(const bf16* __restrict__ src, __half* __restrict__ dst, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __float2half_rn(__bfloat162float(src[i]));
}

// ---- host side ----------------------------------------------------------------------------

}  // namespace

struct LayerMaps {
    bool ready = false;
    CUtensorMap* d_amaps1 = nullptr;    // gate/up: [gate pool, up pool, (ws_gate, ws_up) per model]
    CUtensorMap* d_amaps2 = nullptr;    // down:    [down pool, down pool, (ws_down fp16, same) per model]
    std::vector<__half*> ws_down_f16;   // per model
};

struct TensorMaps {
    std::vector<LayerMaps> layers;
};

bool tc_supported(const moe_ctx* c)
{
    const moe_config& g = c->cfg;
    return g.hidden % 256 == 0 && g.inter % 128 == 0 && g.shared_inter % 128 == 0;
}

void tc_destroy(moe_ctx* c)
{
    if (!c->tmaps) return;
    cudaDeviceSynchronize();
    for (LayerMaps& lm : c->tmaps->layers) {
        if (lm.d_amaps1) cudaFree(lm.d_amaps1);
        if (lm.d_amaps2) cudaFree(lm.d_amaps2);
        for (__half* p : lm.ws_down_f16) if (p) cudaFree(p);
    }
    delete c->tmaps;
    c->tmaps = nullptr;
}

int tc_setup_layer(moe_ctx* c, int layer)
{
    const moe_config& g = c->cfg;
    if (!c->tmaps) {
        c->tmaps = new TensorMaps();
        c->tmaps->layers.resize(g.n_layers);
    }
    LayerMaps& lm = c->tmaps->layers[layer];
    if (lm.ready) return MOE_OK;
    const int M = g.n_models, H = g.hidden, I = g.inter, Is = g.shared_inter;
    const PoolWeights& pw = c->pools[layer];
    std::vector<CUtensorMap> m1(2 + 2 * M), m2(2 + 2 * M);
    memset(m1.data(), 0, m1.size() * sizeof(CUtensorMap));
    memset(m2.data(), 0, m2.size() * sizeof(CUtensorMap));
    bool ok = true;
    const uint64_t S = g.n_slots;
    ok &= make_map(&m1[0], pw.w_gate, S * I, H, 128, false);
    ok &= make_map(&m1[1], pw.w_up, S * I, H, 128, false);
    ok &= make_map(&m2[0], pw.w_down, S * H, I, 128, false);
    m2[1] = m2[0];
    lm.ws_down_f16.assign(M, nullptr);
    for (int m = 0; m < M && ok && Is > 0; ++m) {
        const ModelWeights& mw = c->models[(size_t)layer * M + m];
        ok &= make_map(&m1[2 + 2 * m], mw.ws_gate, Is, H, 128, false);
        ok &= make_map(&m1[3 + 2 * m], mw.ws_up, Is, H, 128, false);
        // fp16 copy of the shared expert's down projection (its activations are fp16 and one MMA takes
        // operands of one type); every bf16 weight of magnitude >= 2^-17 converts exactly
        const size_t n = (size_t)H * Is;
        if (cudaMalloc((void**)&lm.ws_down_f16[m], n * sizeof(__half)) != cudaSuccess) return MOE_ERR_ALLOC;
        bf16_to_fp16_kernel<<<(unsigned)((n + 255) / 256), 256>>>(mw.ws_down, lm.ws_down_f16[m], n);
        ok &= make_map(&m2[2 + 2 * m], lm.ws_down_f16[m], H, Is, 128, true);
        m2[3 + 2 * m] = m2[2 + 2 * m];
    }
    if (!ok) {
        snprintf(c->errbuf, sizeof(c->errbuf), "cuTensorMapEncodeTiled failed for a weight tensor");
        return MOE_ERR_CUDA;
    }
    const size_t bytes = m1.size() * sizeof(CUtensorMap);
    if (cudaMalloc((void**)&lm.d_amaps1, bytes) != cudaSuccess || cudaMalloc((void**)&lm.d_amaps2, bytes) != cudaSuccess)
        return MOE_ERR_ALLOC;
    if (cudaMemcpy(lm.d_amaps1, m1.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(lm.d_amaps2, m2.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess)
        return MOE_ERR_CUDA;
    lm.ready = true;
    return MOE_OK;
}

cudaError_t launch_experts_tc(moe_ctx* c, int layer, const bf16* x_or_xs, const bf16* x_perm, int T, float* y_perm,
                              float* y_shared, const int32_t* shared_dst_rows, cudaStream_t st)
{
    const moe_config& g = c->cfg;
    const LayerMaps& lm = c->tmaps->layers[layer];
    const int H = g.hidden, I = g.inter, Is = g.shared_inter;
    const uint64_t R = (uint64_t)T * g.top_k;
    const bool shared = y_shared != nullptr && Is > 0;

    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncSetAttribute(grouped_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        attr_set = true;
    }
    const uint32_t fmt_bf16 = (1u << 7) | (1u << 10), fmt_fp16 = 0u;

    // B operand maps are rebuilt per call: the activations' addresses and row counts are the call's
    CUtensorMap br128, br16, bs128, bs16;
    bool ok = make_map(&br128, x_perm, R, H, 128, false) && make_map(&br16, x_perm, R, H, 16, false);
    if (shared) ok = ok && make_map(&bs128, x_or_xs, T, H, 128, false) && make_map(&bs16, x_or_xs, T, H, 16, false);
    else { bs128 = br128; bs16 = br16; }
    if (!ok) return cudaErrorInvalidValue;

    GemmParams p1;
    p1.units = c->ws.units1; p1.n_units = c->ws.plan_counts + 2;
    p1.tiles = c->ws.tiles; p1.stiles = c->ws.stiles;
    p1.amaps = lm.d_amaps1;
    p1.k_routed = H; p1.k_shared = H;
    p1.rows_per_slot = I; p1.cb_stride = 128; p1.a1_off = 0;
    p1.out_routed = c->ws.h; p1.out_shared = c->ws.hs; p1.ld_routed = I; p1.ld_shared = Is;
    p1.shared_dst_rows = nullptr;
    p1.idesc_fmt_routed = fmt_bf16; p1.idesc_fmt_shared = fmt_bf16;
    p1.status = c->ws.status;
    p1.stream_weights = (R <= 2048) ? 1 : 0;
    grouped_gemm_kernel<0><<<c->sm_count, kThreads, kSmemBytes, st>>>(p1, br128, br16, bs128, bs16);
    stage_mark(c, st, kEvGateUp);

    CUtensorMap hr128, hr16, hs128, hs16;
    ok = make_map(&hr128, c->ws.h, R, I, 128, false) && make_map(&hr16, c->ws.h, R, I, 16, false);
    if (shared) ok = ok && make_map(&hs128, c->ws.hs, T, Is, 128, true) && make_map(&hs16, c->ws.hs, T, Is, 16, true);
    else { hs128 = hr128; hs16 = hr16; }
    if (!ok) return cudaErrorInvalidValue;
    GemmParams p2 = p1;
    p2.units = c->ws.units2; p2.n_units = c->ws.plan_counts + 3;
    p2.amaps = lm.d_amaps2;
    p2.k_routed = I; p2.k_shared = Is;
    p2.rows_per_slot = H; p2.cb_stride = 256; p2.a1_off = 128;
    p2.out_routed = y_perm; p2.out_shared = y_shared; p2.ld_routed = H; p2.ld_shared = H;
    p2.shared_dst_rows = shared_dst_rows;
    p2.idesc_fmt_routed = fmt_bf16; p2.idesc_fmt_shared = fmt_fp16;
    grouped_gemm_kernel<1><<<c->sm_count, kThreads, kSmemBytes, st>>>(p2, hr128, hr16, hs128, hs16);
    stage_mark(c, st, kEvDown);
    c->launches += 2;
    return cudaGetLastError();
}

}  // namespace faasmoe
