// Internal declarations shared by the translation units of libfaasmoe.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <vector>

#include "faasmoe.h"

namespace faasmoe {

typedef __nv_bfloat16 bf16;

constexpr int kMaxTopK = 8;
constexpr int kMaxExperts = 256;
constexpr int kMaxBins = 8192;       // E * n_tenants
constexpr int kTileRows = 128;       // rows (tokens) of one expert handled by one work unit
constexpr int kDispatchChunk = 256;  // routed rows ranked by one block of the dispatch kernels
constexpr int kAccRowsBg = 224;      // pair shape with background lanes: token rows per accumulator of a wide tile (two per tile)
constexpr int kShortRows = 64;       // pair shape: tiles of at most this many rows may be run by the background lanes
constexpr int kFusedDispatchTokens = 128;        // tokens one router CTA handles
constexpr size_t kFusedDispatchSmem = 128 * 1024; // scratch the router's stage ring offers the dispatch behind it
constexpr int kMaxDevices = 64;      // per-device state of the library (kernel attributes, scratch addresses)

// Per (layer, model) weight pointers, as the kernels see them.
struct ModelWeights {
    const bf16* router_w;       // [E,H]
    const float* router_bias;   // [E] or null
    const bf16* shared_gate_w;  // [H] or null
    const bf16* ws_gate;        // [Is,H]
    const bf16* ws_up;          // [Is,H]
    const bf16* ws_down;        // [H,Is]
    const bf16* rms_w;          // [H]
};

struct PoolWeights {
    const bf16* w_gate;  // [S,I,H]
    const bf16* w_up;    // [S,I,H]
    const bf16* w_down;  // [S,H,I]
};

// One tile of rows that share an expert: rows [row0, row0+nrows) of the activation
// matrix, weights of `slot` (routed: pool slot; shared: model index).
struct Tile {
    int32_t row0;
    int32_t nrows;
    int32_t slot;
    int32_t group;   // expert block (m*B + b) for routed tiles, model for shared tiles
};

// Work unit of the tensor-core grouped GEMM: a tile (>= 0 routed, < 0: shared tile ~tile)
// and a block of weight rows.
struct Unit {
    int32_t tile;
    int32_t colblock;
};

struct TensorMaps;   // defined in experts_tc.cu

// On-demand residency of the routed experts (one layer): all experts are parked in host memory, the pool slots on
// the device are a cache of the experts in use, managed least-recently-used.
struct Residency {
    bool on = false;
    const bf16* h_gate = nullptr;   // host [M*E, I, H]
    const bf16* h_up = nullptr;
    const bf16* h_down = nullptr;   // host [M*E, H, I]
    bf16* p_gate = nullptr;         // device pool [S, I, H] (the arrays registered with moe_set_expert_pool)
    bf16* p_up = nullptr;
    bf16* p_down = nullptr;
    std::vector<int32_t> owner;     // [S] expert in the slot, -1: free
    std::vector<int64_t> last_use;  // [S] call that used the slot last
    std::vector<int32_t> slot_of;   // [M*E] slot of the expert, -1: parked
    int64_t clock = 0;
    int32_t* d_active = nullptr;    // [M*E] device flags of the experts the current batch routes to
    int32_t* h_active = nullptr;    // the same in pinned host memory
};

struct Workspace {
    // routing results
    int32_t* topk_idx = nullptr;   // [T,k]
    float* topk_w = nullptr;       // [T,k]
    float* shared_gate = nullptr;  // [T]
    uint8_t* tie_flag = nullptr;   // [T]
    // dispatch results
    int32_t* perm = nullptr;       // [R]
    int32_t* inv_perm = nullptr;   // [R]
    int32_t* tenant_expert_count = nullptr;  // [Nt*E]
    int32_t* expert_off = nullptr; // [M*E+1]
    int32_t* group_off = nullptr;  // [M*E+1] (largest B is E)
    // dispatch scratch
    int32_t* block_cnt = nullptr;  // [nblk, nbins]
    int32_t* bin_off = nullptr;    // [nbins+1]
    int32_t* dispatch_done = nullptr;  // [1] blocks of the counting kernel that have finished (zero between calls)
    int32_t* tok_block_cnt = nullptr;  // [nblk_tok, M]
    int32_t* model_tok_off = nullptr;  // [M+1]
    int32_t* tok_perm = nullptr;   // [T] tokens sorted by (model, token)
    int32_t* tok_inv = nullptr;    // [T]
    // plan
    Tile* tiles = nullptr;         // routed tiles
    Tile* stiles = nullptr;        // shared-expert tiles
    int32_t* tile_cidx = nullptr;  // [tiles] index of a routed tile inside its class (long / short)
    int32_t* plan_counts = nullptr;  // [16]: n_tiles, n_stiles, n_units1, n_units2, -, -, shared units to spread (2),
                                     //       short units (2), work counters of the two launches (2 words each)
    Unit* units1 = nullptr;        // gate/up GEMM units (shared, then routed)
    Unit* units2 = nullptr;        // down GEMM units
    // the same for the shared expert alone (one model), when it runs beside the router and the dispatch
    Tile* stiles_sh = nullptr;
    int32_t* plan_counts_sh = nullptr;  // [16]
    Unit* units1_sh = nullptr;
    Unit* units2_sh = nullptr;
    // activations
    bf16* x_perm = nullptr;        // [R,H]
    bf16* xs_perm = nullptr;       // [T,H] tokens grouped by model (M > 1 only)
    bf16* h = nullptr;             // [R,I]
    void* hs = nullptr;            // [T,Is] fp16: SwiGLU activations of the shared expert.  fp16 rather than
                                   // bf16 because the 4x wider down-projection sums 4x more rounding errors and
                                   // the gated result enters the output with a weight of ~0.5 instead of ~0.1
    float* y_perm = nullptr;       // [R,H] fp32: un-weighted expert outputs; kept in fp32 because the combine
    float* y_shared = nullptr;     // [T,H]       adds terms of opposite sign and bf16 rounding would not cancel
    bf16* xn = nullptr;            // [T,H] normalised input of a block (stack)
    // staging of the host-buffer entry point
    bf16* x_stage = nullptr;       // [T,H]
    int32_t* tenant_stage = nullptr;  // [T]
    bf16* out_stage = nullptr;     // [T,H]
    // second set of staging buffers: the pipelined host entry point keeps two submissions in flight
    bf16* x_stage2 = nullptr;
    int32_t* tenant_stage2 = nullptr;
    bf16* out_stage2 = nullptr;
    // status
    int32_t* status = nullptr;     // [1] sticky status bits
    int32_t* stats = nullptr;      // [4]
};

}  // namespace faasmoe

struct moe_ctx {
    moe_config cfg;
    int device;
    int sm_count;
    int expert_path;
    int64_t launches;
    int max_tiles, max_stiles, max_units1, max_units2;
    int nblk_rows, nblk_tok, nbins;
    std::vector<faasmoe::PoolWeights> pools;     // [L]
    std::vector<uint8_t> pool_set;               // [L]
    std::vector<faasmoe::ModelWeights> models;   // [L*M]
    std::vector<uint8_t> model_set;              // [L*M]
    faasmoe::ModelWeights* d_models;             // [L*M] device copy
    std::vector<int32_t> h_slot, h_model_of_tenant;
    int32_t* d_slot;              // [M*E]
    int32_t* d_model_of_tenant;   // [Nt]
    int32_t* d_tenant_local;      // [Nt] index of the tenant among the tenants of its model
    faasmoe::Residency res;       // on-demand residency of the routed experts
    int32_t* d_block_table;       // [M*E] block of every expert (load-aware formation), null: blocks of G consecutive experts
    int table_blocks;             // blocks per model of that table
    int32_t* d_bin_base;          // [M+1] first bin of each model (bins = (model, expert, tenant of model))
    int32_t* d_tenants_in_model;  // [M]
    faasmoe::Workspace ws;
    faasmoe::TensorMaps* tmaps;   // TMA descriptors of the tensor-core path (host)
    void* rmaps;                  // TMA descriptors of the tensor-core router
    int route_path;
    int route_lanes2;             // the tensor-core router issues its MMAs from two warps
    int pair_mode_enabled;        // allow the 2-CTA (cta_group::2) shape of the grouped GEMM for long tiles
    int token_major_enabled;      // one-CTA units take the tokens as the M operand of the MMA (up to 256 weight rows per tile)
    int wide_tiles_enabled;       // allow 512-row tiles (two accumulators per weight tile) in the 2-CTA shape
    int head_units_enabled;       // token-major gate/up launch of a layer pass: shared-expert units before the wait
    int fused_dispatch_enabled;   // one-tile batches: the router's CTA also runs the dispatch and the work plan
    int background_enabled;       // pair shape: short tiles are run by a second set of lanes beside the long ones
    int dispatch_private;         // 0: shared orchestrator (one request per expert block), 1: private orchestrators
                                  // (one request per tenant and block): invocation statistics and tile formation
    int early_shared_enabled;     // one model: run the shared expert on a second stream beside router and dispatch
                                  // (1: batches of the 2-CTA shape, 2: every batch)
    int early_shared_sms;         // SMs the shared expert's CTA pairs may take while they run beside other kernels
    cudaStream_t copy_in, copy_out;   // streams of the pipelined host entry point (H2D of the next call, D2H of the last)
    cudaEvent_t ev_in[2], ev_done[2], ev_out[2];   // per staging slot: inputs landed, layer done, outputs landed
    int64_t submitted;            // submissions so far (ticket of the next one)
    int64_t waited[2];            // last ticket of each slot whose outputs are known to have landed
    cudaStream_t side;            // second stream of the layer pass
    cudaEvent_t ev_fork, ev_join; // order between the caller's stream and the second one
    bool timing;                  // record an event after every stage (moe_layer_forward_timed)
    cudaEvent_t ev[8];
    char errbuf[256];
};

// stage boundaries of one layer pass
enum { kEvBegin = 0, kEvRoute, kEvDispatch, kEvPlan, kEvGateUp, kEvDown, kEvCombine, kEvCount };

static inline void stage_mark(moe_ctx* c, cudaStream_t st, int i)
{
    if (c->timing) cudaEventRecord(c->ev[i], st);
}

namespace faasmoe {

// Programmatic dependent launch: the kernels of a layer pass are launched so that each may be set up (block
// scheduling, barrier initialisation, TMEM allocation) while its predecessor in the stream is still running.  Every
// such kernel calls pdl_wait() before it reads anything a predecessor wrote, and every block passes through it
// before it exits, so completion of a kernel implies completion of all earlier ones.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg;
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// --- launchers (each returns a cudaError_t from the launch) -------------------------------

cudaError_t launch_route(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                         float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st);

cudaError_t launch_dispatch(moe_ctx* c, const bf16* x, const int32_t* topk_idx, const int32_t* tenant_id, int T, int G,
                            int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off,
                            int32_t* group_off, bf16* x_perm, cudaStream_t st, bool with_plan = false,
                            bool plan_shared = false, bool* plan_done = nullptr);

cudaError_t launch_route_fma(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                             float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st);
struct SmallDispatchArgs;
// fused: arguments of the one-block dispatch that the router's CTA runs behind its top-k step (one-tile batch of one
// model; fused_smem bytes of scratch), or null
cudaError_t launch_route_tc(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int32_t* topk_idx,
                            float* topk_w, float* shared_gate, uint8_t* tie_flag, cudaStream_t st,
                            const SmallDispatchArgs* fused = nullptr, size_t fused_smem = 0);
// Router, then -- where one CTA routes the whole batch -- dispatch and work plan in the same launch.  *fused tells the
// caller whether the dispatch has been done (and *plan_done whether the plan has); if not, launch_dispatch follows.
cudaError_t launch_route_dispatch(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, int G,
                                  int32_t* topk_idx, float* topk_w, float* shared_gate, uint8_t* tie_flag, int32_t* perm,
                                  int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off, int32_t* group_off,
                                  bf16* x_perm, cudaStream_t st, bool plan_shared, bool* fused, bool* plan_done);
bool route_tc_supported(const moe_ctx* c);
void route_tc_destroy(moe_ctx* c);

// Sorts tokens by (model, token) into ws.tok_perm / tok_inv / model_tok_off and gathers ws.xs_perm (M > 1).
cudaError_t launch_token_sort(moe_ctx* c, const bf16* x, const int32_t* tenant_id, int T, cudaStream_t st);

struct PlanArgs;
PlanArgs make_plan_args(moe_ctx* c, int T, int G, bool with_shared);
size_t plan_smem_ints(const moe_ctx* c, int G);

// Builds the tile lists (and the unit lists of the tensor-core path) from expert_off.
cudaError_t launch_plan(moe_ctx* c, const int32_t* expert_off, int T, int G, bool with_shared, cudaStream_t st);
// unit lists of the shared expert alone (one model) and how many units they hold
cudaError_t launch_plan_shared(moe_ctx* c, int T, cudaStream_t st);
void shared_unit_counts(moe_ctx* c, int T, int* n_units1, int* n_units2);

cudaError_t launch_experts_fma(moe_ctx* c, int layer, const bf16* x_or_xs, const bf16* x_perm, int T, float* y_perm,
                               float* y_shared, const int32_t* shared_dst_rows, cudaStream_t st);

cudaError_t launch_experts_tc(moe_ctx* c, int layer, const bf16* x_or_xs, const bf16* x_perm, const int32_t* perm, int T,
                              float* y_perm, float* y_shared, const int32_t* shared_dst_rows, cudaStream_t st,
                              bool shared_only = false, bool tokens_ready = false);

cudaError_t launch_combine(moe_ctx* c, const float* y_perm, const int32_t* inv_perm, const float* topk_w,
                           const float* y_shared, const float* shared_gate, const bf16* residual, int T, bf16* out,
                           cudaStream_t st);

cudaError_t launch_rmsnorm(moe_ctx* c, int layer, const bf16* x, const int32_t* tenant_id, int T, bf16* xn,
                           cudaStream_t st);

// tensor-core path set-up / tear-down (TMA descriptors); returns MOE_* status
int tc_setup_layer(moe_ctx* c, int layer);
void tc_destroy(moe_ctx* c);
bool tc_supported(const moe_ctx* c);
bool tc_pair_mode(const moe_ctx* c, int T);      // long tiles: two CTAs share a token tile
bool tc_wide_mode(const moe_ctx* c, int T);      // pair shape with tiles of up to 2 * kAccRows rows
bool tc_background_mode(const moe_ctx* c, int T);   // pair shape with background lanes for the short tiles
bool tc_token_major(const moe_ctx* c, int T);    // one-CTA shape with the tokens as the M operand

// Few tokens of one model: the routed gate/up units read the tokens in place, no permuted copy is needed.
static inline bool tc_direct_mode(const moe_ctx* c, int T)
{
    return tc_supported(c) && !tc_pair_mode(c, T) && T <= 128 && c->cfg.n_models == 1;
}

}  // namespace faasmoe
