// Gating network on the tensor cores (paper Sec. 2.1: the gate scores every expert and selects
// the top-k per token).  One CTA scores 128 tokens against the router of one tenant model: the
// tokens are the M operand of tcgen05.mma (one TMEM lane per token), the router rows the N operand
// (E rows, padded to a multiple of 16, followed by 16 rows for the shared expert's gate vector).
// With several models the grid is (token tiles x models) and a CTA writes the results of those
// tokens of its tile that belong to its model.  Two warps issue the MMAs, even and odd K stages
// into an accumulator each.  The epilogue is one thread per token: it adds the two accumulators and
// the router bias (fetched while the MMAs run) and does the fp32 softmax and the top-k in registers.
#include <cstring>

#include "internal.h"
#include "dispatch_small.cuh"
#include "tc_ptx.cuh"

namespace faasmoe {

namespace {

using namespace tc;

constexpr int kRMaxStages = 16;
constexpr int kRBK = 64;
constexpr int kRTokens = 128;
constexpr int kRABytes = kRTokens * kRBK * 2;          // 16 KB of tokens per stage
constexpr int kRMaxN = 256;                            // router rows of all models, padded
constexpr int kRTileBudget = 192 * 1024;               // shared memory for the pipeline stages
static_assert(kFusedDispatchSmem <= (size_t)kRTileBudget, "the dispatch behind the router uses the stage ring as scratch");
constexpr int kRSmemBytes = kRTileBudget + kRABytes /* a short token tile is read as 128 rows */ + 1024 + 512;
constexpr int kRThreads = 288;                         // warp 0: TMA (tokens), 1: MMA, 2..5: epilogue, 6 / 7: TMA (routers / gates),
                                                       // 8: second MMA lane
constexpr int kRMaxE = 64;                             // logits one thread keeps in registers

struct RouteParams {
    const bf16* x;
    const int32_t* tenant_id;
    int T, H, E, Epad, k, n_tenants, n_models;
    const int32_t* model_of_tenant;
    const ModelWeights* models;
    int gate_mma;                  // 1: the gate logit of model m is accumulator column gate_col + m*16
    int gate_col;                  // first gate column: right after the router columns when one MMA covers both
    int gate_merged;               // 1: router rows and gate rows are one N operand (n_models * (Epad + 16) <= 256)
    int lanes2;                    // 1: two warps issue the MMAs, even and odd stages into accumulators of their own
                                   // (TMEM columns 0.. and 256..) that the epilogue adds up
    int per_model;                 // 1: blockIdx.y is a model; the CTA computes that model's logits only and writes the
                                   // results of the tile's tokens that belong to it
    int group;                     // stages handed back to the producer per commit (divides n_stages)
    int kb;                        // slices of 64 K elements per stage (1, 2 or 4): a wait, a fence and a commit per stage
                                   // cost the MMA lane as much as several of these narrow MMAs
    int bg_bytes;                  // router rows + gate rows of one slice
    int a_bytes, b_bytes, stage_bytes, n_stages;   // pipeline geometry: small batches take more, smaller stages
    int32_t* topk_idx;
    float* topk_w;
    float* shared_gate;
    uint8_t* tie_flag;
    int32_t* status;
};

constexpr int kRMaxModels = 4;

// TMA descriptors, passed in kernel parameter space
struct RouteMaps {
    CUtensorMap x;                       // tokens [T,H], box a_rows
    CUtensorMap r[kRMaxModels];          // router_w [E,H] of each model, box Epad rows
    CUtensorMap g[kRMaxModels];          // shared_gate_w [1,H] of each model, box 16 rows (15 read as zero)
};

__device__ __forceinline__ float dot8f(const uint4& a, const uint4& b, float acc)
{
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
    }
    return acc;
}

// (a call, not inlined: the registers of the dispatch stay out of the router's own allocation)
__device__ __noinline__ void dispatch_behind_router(const SmallDispatchArgs& fd, int32_t* scratch)
{
    dispatch_small_body(fd, scratch);
}

__global__ void __launch_bounds__(kRThreads, 1)
route_tc_kernel(const RouteParams p, const __grid_constant__ RouteMaps maps, const __grid_constant__ SmallDispatchArgs fd)
{
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t bars = smem_base + kRTileBudget + kRABytes;
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kRMaxStages, bar_tfull = bars + 16 * kRMaxStages;
    const int kRStages = p.n_stages;
    const uint32_t gmask = (uint32_t)p.group - 1, gshift = p.group == 4 ? 2u : (p.group == 2 ? 1u : 0u);      // group: 1, 2 or 4
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * kRTokens;
    const int ksteps = p.H / (kRBK * p.kb);        // stages to go through
    const int m0 = p.per_model ? (int)blockIdx.y : 0;       // first model and number of models of this CTA
    const int nm = p.per_model ? 1 : p.n_models;
    const int N = nm * p.Epad;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_tfull, p.lanes2 ? 2 : 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    // Set-up above overlaps the previous kernel; its results are read from here on.  The producer lanes of the router
    // and gate rows read static weights only: they fill the first stages while the others still wait.
    if (!(warp == 6 || warp == 7)) pdl_wait();
    pdl_launch_dependents();

    if (warp == 0 || warp == 6 || warp == 7) {
        // three producer lanes (tokens / routers / gates) in three warps, so that the TMA instructions of one stage
        // are issued side by side (a tile load costs its issuing lane about 140 cycles, the barrier handshake about
        // 290; lanes of one warp would run their branches one after the other); the token lane also posts the
        // byte count
        const int role = warp == 0 ? 0 : warp - 5;
        if (lane == 0 && (role < 2 || p.gate_mma)) {
            uint32_t stage = 0, phase = 0, armed = 0, armed_phase = 0;
            bool ok = true;
            const uint64_t keep = l2_evict_last();      // router weights and tokens are read again soon
            for (int ks = 0; ks < ksteps; ++ks) {
                if ((stage & gmask) == 0 &&
                    !mbar_wait(bar_empty + 8 * (stage >> gshift), phase ^ 1, &s_abort, p.status)) { ok = false; break; }
                // stage: kb token slices, then kb slices of (router rows, gate rows)
                const uint32_t sa = smem_base + stage * p.stage_bytes, sb = sa + p.kb * p.a_bytes;
                const uint32_t full = bar_full + 8 * stage;
                armed |= 1u << stage;
                armed_phase = (armed_phase & ~(1u << stage)) | (phase << stage);
                if (role == 0) {
                    mbar_expect_tx(full, p.kb * (p.a_bytes + N * kRBK * 2 + (p.gate_mma ? nm * 16 * kRBK * 2 : 0)));
                    for (int a = 0; a < p.kb; ++a) tma_load_2d_hint(sa + a * p.a_bytes, &maps.x, full, (ks * p.kb + a) * kRBK, t0, keep);
                } else if (role == 1) {
                    for (int a = 0; a < p.kb; ++a)
                        for (int m = 0; m < nm; ++m)
                            tma_load_2d_hint(sb + a * p.bg_bytes + m * p.Epad * kRBK * 2, &maps.r[m0 + m], full, (ks * p.kb + a) * kRBK, 0, keep);
                } else {
                    for (int a = 0; a < p.kb; ++a)
                        for (int m = 0; m < nm; ++m)
                            tma_load_2d_hint(sb + a * p.bg_bytes + p.b_bytes + m * 16 * kRBK * 2, &maps.g[m0 + m], full, (ks * p.kb + a) * kRBK, 0,
                                             keep);
                }
                if (++stage == kRStages) { stage = 0; phase ^= 1; }
            }
            if (!ok && role == 0)
                for (int s = 0; s < kRStages; ++s)
                    if (armed & (1u << s)) mbar_wait(bar_full + 8 * s, (armed_phase >> s) & 1u, &s_abort, p.status);
        }
        __syncwarp();
    } else if (warp == 1 || warp == 8) {
        // The MMAs of a stage cost their issuing lane more than the tensor pipe: with two lanes (in two warps) the
        // stages alternate between them.
        const int mine = warp == 1 ? 0 : 1;
        if (lane == 0 && (mine == 0 || p.lanes2)) {
            uint32_t stage = 0, phase = 0;
            const uint32_t tmem_acc = tmem_base + (uint32_t)mine * 256u;
            // a tcgen05.mma costs its issuing lane about 100 cycles whatever its width, a commit about 200: the gate
            // rows ride in the router's MMA when they fit, and stages go back to the producer in groups
            const int n_main = p.gate_merged ? N + nm * 16 : N;
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_main >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_g = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(nm * 16 >> 3) << 17) | ((128u >> 4) << 24);
            bool ok = true;
            const uint32_t a_step = (uint32_t)p.a_bytes >> 4, bg_step = (uint32_t)p.bg_bytes >> 4;
            const uint32_t b_off = (uint32_t)(p.kb * p.a_bytes) >> 4, g_off = (uint32_t)p.b_bytes >> 4;
            const bool two_mmas = p.gate_mma && !p.gate_merged;
            uint32_t acc = 0;                   // the first MMA overwrites the accumulators
            for (int ks = 0; ks < ksteps; ++ks) {
                if (p.lanes2 && (ks & 1) != mine) {
                    if (++stage == kRStages) { stage = 0; phase ^= 1; }
                    continue;
                }
                if (!mbar_wait(bar_full + 8 * stage, phase, &s_abort, p.status)) { ok = false; break; }
                tc_fence_after();
                // (this lane is alone in its warp and pays for every instruction: descriptors from 32-bit words)
                uint32_t lo_a = smem_desc_lo(smem_base + stage * p.stage_bytes);
                uint32_t lo_b = lo_a + b_off;
                for (int a = 0; a < p.kb; ++a) {
                    const uint32_t lo_g = lo_b + g_off;
#pragma unroll
                    for (int kk = 0; kk < kRBK / 16; ++kk) {
                        umma_bf16(tmem_acc, smem_desc_pack(lo_a + 2 * kk), smem_desc_pack(lo_b + 2 * kk), idesc, acc);
                        if (two_mmas) umma_bf16(tmem_acc + p.gate_col, smem_desc_pack(lo_a + 2 * kk), smem_desc_pack(lo_g + 2 * kk), idesc_g, acc);
                        acc = 1;
                    }
                    lo_a += a_step; lo_b += bg_step;
                }
                if ((stage & gmask) == gmask) umma_commit(bar_empty + 8 * (stage >> gshift));
                if (++stage == kRStages) { stage = 0; phase ^= 1; }
            }
            if (ok) umma_commit(bar_tfull);
        }
        __syncwarp();
    } else {
        // ---- epilogue warps: thread <-> token (TMEM lane) ----
        const int quarter = warp & 3;
        const int t = t0 + quarter * 32 + lane;
        bool valid = t < p.T;
        bool bad = false;
        int model = 0;
        if (valid) {
            int u = p.tenant_id[t];
            if (u < 0 || u >= p.n_tenants) { bad = true; u = 0; }
            model = p.model_of_tenant[u];
            if (p.per_model && model != m0) valid = false;      // another CTA of this tile has that model
        }
        // shared-expert gate, overlapped with the MMA pipeline: each thread walks its own token's row
        // (independent 16-byte loads, four accumulators), so no cross-lane traffic is needed
        float gate = 0.5f;
        if (p.shared_gate && valid && !p.gate_mma) {
            const bf16* sg = p.models[model].shared_gate_w;
            if (sg) {
                const uint4* xv = reinterpret_cast<const uint4*>(p.x + (size_t)t * p.H);
                const uint4* wv = reinterpret_cast<const uint4*>(sg);
                const int hv = p.H >> 3;
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
                int v = 0;
                for (; v + 4 <= hv; v += 4) {
                    const uint4 x0 = __ldg(xv + v), x1 = __ldg(xv + v + 1), x2 = __ldg(xv + v + 2), x3 = __ldg(xv + v + 3);
                    a0 = dot8f(x0, __ldg(wv + v), a0);
                    a1 = dot8f(x1, __ldg(wv + v + 1), a1);
                    a2 = dot8f(x2, __ldg(wv + v + 2), a2);
                    a3 = dot8f(x3, __ldg(wv + v + 3), a3);
                }
                for (; v < hv; ++v) a0 = dot8f(__ldg(xv + v), __ldg(wv + v), a0);
                gate = 1.f / (1.f + expf(-((a0 + a1) + (a2 + a3))));
            }
        }
        // this token's router bias (-inf beyond the last expert) is fetched while the MMAs run
        float zb[kRMaxE];
        {
            const float* rb = valid ? p.models[model].router_bias : nullptr;
#pragma unroll
            for (int e = 0; e < kRMaxE; ++e) zb[e] = e < p.E ? (rb ? __ldg(rb + e) : 0.f) : -INFINITY;
        }
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull, 0, &s_abort, p.status));
        if (ok) {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            // logits of this token's model: the column range depends on the model, the TMEM load is
            // warp-wide, so every model's columns are loaded and each thread keeps its own
            float z[kRMaxE];
#pragma unroll
            for (int e = 0; e < kRMaxE; ++e) z[e] = -INFINITY;
            for (int mi = 0; mi < nm; ++mi) {
                const int m = m0 + mi;
#pragma unroll
                for (int c = 0; c < kRMaxE / 16; ++c) {
                    if (c * 16 < p.Epad) {                                // warp-uniform
                        uint32_t r[16], r2[16];
                        tmem_ld16(taddr + mi * p.Epad + c * 16, r);
                        if (p.lanes2) tmem_ld16(taddr + 256 + mi * p.Epad + c * 16, r2);   // the second lane's share of the sum over K
                        tmem_ld_wait();
                        if (m == model) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                z[c * 16 + j] = __uint_as_float(r[j]) + zb[c * 16 + j];
                                if (p.lanes2) z[c * 16 + j] += __uint_as_float(r2[j]);
                            }
                        }
                    }
                }
            }
            if (p.gate_mma && p.shared_gate) {
                for (int mi = 0; mi < nm; ++mi) {
                    const int m = m0 + mi;
                    uint32_t r[16];
                    tmem_ld16(taddr + p.gate_col + mi * 16, r);
                    tmem_ld_wait();
                    float gl = __uint_as_float(r[0]);
                    if (p.lanes2) {
                        tmem_ld16(taddr + 256 + p.gate_col + mi * 16, r);
                        tmem_ld_wait();
                        gl += __uint_as_float(r[0]);
                    }
                    if (m == model && valid && p.models[m].shared_gate_w) gate = 1.f / (1.f + expf(-gl));
                }
            }
            if (valid) {
                // Softmax is monotone, so the ranking is done on the logits themselves; the
                // probabilities are exp2((z - zmax) * log2 e) / sum.  Four independent chains keep
                // the one warp per scheduler busy.
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                for (int e = 0; e < kRMaxE; e += 4) {
                    m0 = fmaxf(m0, z[e]); m1 = fmaxf(m1, z[e + 1]); m2 = fmaxf(m2, z[e + 2]); m3 = fmaxf(m3, z[e + 3]);
                }
                const float zmax = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
                const float kLog2e = 1.4426950408889634f;
                float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
                for (int e = 0; e < kRMaxE; e += 4) {
                    d0 += exp2f((z[e] - zmax) * kLog2e);     d1 += exp2f((z[e + 1] - zmax) * kLog2e);
                    d2 += exp2f((z[e + 2] - zmax) * kLog2e); d3 += exp2f((z[e + 3] - zmax) * kLog2e);
                }
                const float inv_den = 1.f / ((d0 + d1) + (d2 + d3));
                const int rounds = (p.k < p.E) ? p.k + 1 : p.k;
                float prev = 0.f;
                uint8_t flag = 0;
                uint32_t taken_lo = 0, taken_hi = 0;      // experts already selected (a bit mask: writing to
                                                          // z[bi] would be a data-dependent register index)
                for (int j = 0; j < rounds; ++j) {
                    // arg-max with ties to the lower id: each chain scans ids of one residue class in
                    // ascending order, the merge prefers the larger value, then the smaller id
                    float v0 = -INFINITY, v1 = -INFINITY, v2 = -INFINITY, v3 = -INFINITY;
                    int i0 = 0, i1 = 1, i2 = 2, i3 = 3;
#pragma unroll
                    for (int e = 0; e < kRMaxE; e += 4) {
                        const uint32_t tk = (e < 32) ? taken_lo : taken_hi;
                        if (z[e] > v0 && !(tk & (1u << (e & 31)))) { v0 = z[e]; i0 = e; }
                        if (z[e + 1] > v1 && !(tk & (1u << ((e + 1) & 31)))) { v1 = z[e + 1]; i1 = e + 1; }
                        if (z[e + 2] > v2 && !(tk & (1u << ((e + 2) & 31)))) { v2 = z[e + 2]; i2 = e + 2; }
                        if (z[e + 3] > v3 && !(tk & (1u << ((e + 3) & 31)))) { v3 = z[e + 3]; i3 = e + 3; }
                    }
                    if (v1 > v0 || (v1 == v0 && i1 < i0)) { v0 = v1; i0 = i1; }
                    if (v3 > v2 || (v3 == v2 && i3 < i2)) { v2 = v3; i2 = i3; }
                    if (v2 > v0 || (v2 == v0 && i2 < i0)) { v0 = v2; i0 = i2; }
                    const int bi = i0;
                    const float bv = exp2f((v0 - zmax) * kLog2e) * inv_den;
                    if (j > 0 && (prev - bv) < 1e-5f * prev) flag = 1;
                    prev = bv;
                    if (j < p.k) {
                        p.topk_idx[(size_t)t * p.k + j] = bad ? j : bi;
                        p.topk_w[(size_t)t * p.k + j] = bad ? 0.f : bv;
                    }
                    if (bi < 32) taken_lo |= 1u << bi; else taken_hi |= 1u << (bi - 32);
                }
                if (p.tie_flag) p.tie_flag[t] = flag;
                if (p.shared_gate) p.shared_gate[t] = bad ? 0.f : gate;
                if (bad) atomicOr(p.status, MOE_DEV_BAD_TENANT);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    // One-tile batch of one model: this block holds every routed row, so it goes on to batch them per expert block
    // (Sec. 3, Sec. 4.1) and to lay out the experts' work, instead of a kernel of its own doing so after a launch and a
    // round trip through global memory.  The pipeline stages are free by now (every tile load was consumed by an MMA
    // that the top-k step waited for) and serve as scratch.  Not after a wait ran out: copies may still be in flight.
    if (fd.enabled && !s_abort)
        dispatch_behind_router(fd, reinterpret_cast<int32_t*>(smem_dyn + (smem_base - smem_u32(smem_dyn))));
}

struct RouterMaps {
    std::vector<RouteMaps> maps;          // per layer (the token map is filled per call)
    std::vector<int> ready;
    std::vector<int> gate_mma;            // per layer: every model has a gate vector
};

}  // namespace

bool route_tc_supported(const moe_ctx* c)
{
    const moe_config& g = c->cfg;
    const int epad = (g.n_experts + 15) & ~15;
    return g.n_experts <= kRMaxE && g.n_models <= kRMaxModels && g.n_models * epad <= kRMaxN && g.hidden % kRBK == 0;
}

void route_tc_destroy(moe_ctx* c)
{
    RouterMaps* rm = reinterpret_cast<RouterMaps*>(c->rmaps);
    if (!rm) return;
    delete rm;
    c->rmaps = nullptr;
}

cudaError_t launch_route_tc(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                            float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st,
                            const SmallDispatchArgs* fused, size_t fused_smem)
{
    const moe_config& g = c->cfg;
    const int M = g.n_models, E = g.n_experts, H = g.hidden;
    const int epad = (E + 15) & ~15;
    if (!c->rmaps) {
        RouterMaps* rm = new RouterMaps();
        rm->maps.resize(g.n_layers);
        rm->ready.assign(g.n_layers, 0);
        rm->gate_mma.assign(g.n_layers, 0);
        c->rmaps = rm;
    }
    RouterMaps* rm = reinterpret_cast<RouterMaps*>(c->rmaps);
    if (!rm->ready[layer]) {
        RouteMaps& mp = rm->maps[layer];
        memset(&mp, 0, sizeof(mp));
        int gate_mma = 1;
        for (int m = 0; m < M; ++m) {
            const ModelWeights& mw = c->models[(size_t)layer * M + m];
            if (!make_map(&mp.r[m], mw.router_w, E, H, epad, false)) return cudaErrorInvalidValue;
            if (!mw.shared_gate_w) gate_mma = 0;
        }
        for (int m = 0; m < M && gate_mma; ++m)
            if (!make_map(&mp.g[m], c->models[(size_t)layer * M + m].shared_gate_w, 1, H, 16, false)) gate_mma = 0;
        rm->gate_mma[layer] = gate_mma;
        rm->ready[layer] = 1;
    }
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static bool attr_set[kMaxDevices] = {false};
    if (c->device < 0 || c->device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[c->device]) {
        const cudaError_t ea = cudaFuncSetAttribute(route_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRSmemBytes);
        if (ea != cudaSuccess) return ea;
        attr_set[c->device] = true;
    }
    // token tile: only as many rows as the batch has (the MMA still reads 128 rows; the lanes of the
    // rows that were not loaded are never looked at)
    const int a_rows = T >= kRTokens ? kRTokens : ((T + 7) & ~7);
    RouteMaps& mp = rm->maps[layer];
    if (!make_map(&mp.x, x, T, H, a_rows, false)) return cudaErrorInvalidValue;
    RouteParams p;
    p.x = x; p.tenant_id = tenant_id; p.T = T; p.H = H; p.E = E; p.Epad = epad; p.k = g.top_k;
    p.n_tenants = g.n_tenants; p.n_models = M; p.model_of_tenant = c->d_model_of_tenant;
    p.models = c->d_models + (size_t)layer * M;
    p.gate_mma = (shared_gate && rm->gate_mma[layer]) ? 1 : 0;
    p.topk_idx = topk_idx; p.topk_w = topk_w; p.shared_gate = shared_gate; p.tie_flag = tie_flag;
    p.status = c->ws.status;
    p.a_bytes = (a_rows * kRBK * 2 + 1023) & ~1023;
    // several models: a CTA per (token tile, model) computes that model's logits only (4x the CTAs for a quarter of
    // the operand bytes and MMA columns each; a token needs the logits of its own model alone)
    p.per_model = M > 1 ? 1 : 0;
    const int Mc = p.per_model ? 1 : M;             // models per CTA
    p.b_bytes = (Mc * epad * kRBK * 2 + 1023) & ~1023;
    p.bg_bytes = p.b_bytes + (p.gate_mma ? ((Mc * 16 * kRBK * 2 + 1023) & ~1023) : 0);
    const int slice_bytes = p.a_bytes + p.bg_bytes;
    p.kb = 1;
    for (int kb = 4; kb > 1; kb >>= 1)
        if ((H / kRBK) % kb == 0 && kRTileBudget / (kb * slice_bytes) >= 3) { p.kb = kb; break; }
    p.stage_bytes = p.kb * slice_bytes;
    p.n_stages = kRTileBudget / p.stage_bytes;
    if (p.n_stages > kRMaxStages) p.n_stages = kRMaxStages;
    p.group = p.n_stages >= 8 ? 4 : (p.n_stages >= 4 ? 2 : 1);
    // the gate rows follow the router rows in shared memory (b_bytes has no padding: Epad is a multiple of 16)
    p.gate_merged = (p.gate_mma && Mc * (epad + 16) <= kRMaxN && p.b_bytes == Mc * epad * kRBK * 2) ? 1 : 0;
    // two MMA lanes unless the gate rows need an accumulator region of their own; each lane hands back its own stages
    p.lanes2 = ((!p.gate_mma || p.gate_merged) && H / (kRBK * p.kb) >= 2 && c->route_lanes2) ? 1 : 0;
    if (p.lanes2) p.group = 1;
    p.n_stages -= p.n_stages % p.group;
    p.gate_col = p.gate_merged ? Mc * epad : kRMaxN;
    SmallDispatchArgs fd;
    memset(&fd, 0, sizeof(fd));
    if (fused) {
        // (the caller offers the dispatch only for a batch that one CTA routes)
        if (T > kRTokens || p.per_model || fused_smem > (size_t)kRTileBudget) return cudaErrorInvalidValue;
        fd = *fused;
        fd.enabled = 1;
    }
    launch_pdl(route_tc_kernel, dim3((T + kRTokens - 1) / kRTokens, p.per_model ? M : 1), dim3(kRThreads), kRSmemBytes, st, p, mp, fd);
    c->launches += 1;
    return cudaGetLastError();
}

}  // namespace faasmoe
