/*
 * faasmoe.h -- C ABI of the B200 (sm_100a) multi-tenant Mixture-of-Experts layer.
 *
 * The layer is the one FaaSMoE serves as a shared pool of stateless expert
 * functions for many tenants: gating and top-k selection (paper Sec. 2.1), the
 * grouping of the routed tokens into one request per expert block (Sec. 3,
 * Sec. 4.1), expert execution on the assigned tokens (Sec. 3), and the
 * aggregation of expert outputs per token (Sec. 3, Sec. 4.2).  The paper's
 * expert-block granularity (G experts per function, Sec. 3 / Sec. 5) is a
 * partition parameter of the expert work; it never changes a result.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless its comment says "host".
 *  - bf16 tensors are passed as `const void*` (16-bit elements, row-major).
 *  - The caller owns every buffer it passes.  Weight buffers are used in
 *    place (no copy is made): they must stay valid and unchanged while any
 *    call that uses them may still run.
 *  - The context owns only its workspace, its tables and its TMA descriptors.
 *  - `stream` is a cudaStream_t passed as `void*` (NULL = default stream).
 *    No call synchronises the stream unless stated.
 *  - Every call returns an int status: MOE_OK (0) or a negative MOE_ERR_*.
 *    Errors the host can detect return before anything is launched.
 *    Data-dependent errors (an id out of range inside a device buffer, a
 *    bounded device-side wait that ran out) set bits in a sticky device
 *    status word, never fault, and are read with moe_last_status().
 *  - Activation and output buffers (x, x_perm, y_perm, y_shared, out, x_inout and the
 *    debug buffers) must be 16-byte aligned: they are accessed with 16-byte vectors and
 *    TMA tiles.  A misaligned pointer returns MOE_ERR_SHAPE and launches nothing.
 *  - Shapes: hidden, inter and shared_inter must be multiples of 128;
 *    1 <= top_k <= min(n_experts, 8); n_experts <= 256.
 *  - One context serves one device (the device current at moe_create) and
 *    one stream at a time: calls on one context must not overlap on the GPU,
 *    because they share its workspace.
 */
#ifndef FAASMOE_H
#define FAASMOE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_ctx moe_ctx;

enum {
    MOE_OK = 0,
    MOE_ERR_NULL = -1,        /* a required pointer is NULL */
    MOE_ERR_SHAPE = -2,       /* a size or id is out of range (T > max_tokens, bad layer/model, ...) */
    MOE_ERR_G = -3,           /* G < 1 or G > n_experts */
    MOE_ERR_STATE = -4,       /* weights for the requested layer/model were not set */
    MOE_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed (see moe_strerror) */
    MOE_ERR_ALLOC = -6,       /* workspace allocation failed */
    MOE_ERR_UNSUPPORTED = -7  /* the shape is outside what the kernels support */
};

/* bits of the device status word */
enum {
    MOE_DEV_BAD_TENANT = 1,   /* tenant id outside [0, n_tenants): the token's output is zero */
    MOE_DEV_BAD_EXPERT = 2,   /* expert id outside [0, n_experts) in a caller-supplied topk_idx */
    MOE_DEV_TIMEOUT = 8       /* a bounded wait inside a kernel ran out; outputs are invalid */
};

/* moe_set_option: which kernels run the expert FFNs (MOE_OPT_EXPERT_PATH) and the router
 * (MOE_OPT_ROUTE_PATH).  AUTO takes the tcgen05 kernels whenever the shape allows
 * (experts: hidden % 256 == 0; router: n_experts <= 64 and n_models * ceil16(n_experts) <= 256),
 * FMA forces the CUDA-core kernels, TCGEN05 fails with MOE_ERR_UNSUPPORTED if not possible. */
enum { MOE_PATH_AUTO = 0, MOE_PATH_FMA = 1, MOE_PATH_TCGEN05 = 2 };
enum { MOE_DISPATCH_SHARED = 0, MOE_DISPATCH_PRIVATE = 1 };
enum { MOE_OPT_EXPERT_PATH = 1, MOE_OPT_ROUTE_PATH = 2,
       MOE_OPT_PAIR_MODE = 3, /* 1 (default): batches of more than 64 tokens use the 2-CTA tcgen05 shape; 0: never;
                                 2: every batch */
       MOE_OPT_TOKEN_MAJOR = 5, /* 1 (default): batches outside the 2-CTA shape (at most 64 tokens) run their expert tiles with the tokens
                                   as the M operand of the MMA and the weight rows as N; 0: weight rows as M.  Results
                                   are bit-identical (the accumulation order over K is the same). */
       MOE_OPT_WIDE_TILES = 4, /* 1 (default; 2 means the same): the 2-CTA shape uses expert tiles of up to 512 rows whose
                                 two 256-column accumulators are fed from one weight tile; 0: tiles of at most 256
                                 rows.  Results are bit-identical either way. */
       MOE_OPT_EARLY_SHARED = 6, /* one model with a shared expert, moe_layer_forward and the calls built on it: the
                                    shared expert's two launches go to a second stream of the context, beside the
                                    router and the dispatch; the combine waits for both.  1 (default): batches of
                                    more than 64 tokens; 2: every batch; 0: never.  Results are bit-identical.
                                    With several models the second stream groups the tokens by model (the input
                                    of the shared experts) beside the router and the dispatch, unless 0. */
       MOE_OPT_EARLY_SHARED_SMS = 7, /* SMs that the shared expert's CTA pairs may hold while they run beside other
                                       kernels (batches of more than 64 tokens; default: no limit) */
       MOE_OPT_DISPATCH_MODE = 9, /* orchestrator placement (Sec. 4.2, strategies FaaSMoE-Shared and FaaSMoE-Private;
                                     Sec. 5 on orchestrator placement).  MOE_DISPATCH_SHARED (default): one orchestrator
                                     batches across tenants -- all rows that reach an expert block form one invocation
                                     and the rows of an expert are tiled whoever owns them.  MOE_DISPATCH_PRIVATE: every
                                     tenant's orchestrator batches only its own tokens -- an invocation is a (tenant,
                                     block) pair with rows, and no tile of expert work spans two tenants (more, smaller
                                     tiles; an expert's weights are fetched once per tenant that uses it).  The
                                     permutation, the offset tables and every output bit are the same in both modes
                                     (rows are ordered (model, expert, tenant, token) either way); what changes is the
                                     invocation count reported by moe_last_status and the cost of moe_experts.
                                     In private mode moe_experts takes the (expert, tenant) boundaries from the last
                                     moe_dispatch that the same context ran in private mode: set the mode before the
                                     dispatch, not between dispatch and experts. */
       MOE_OPT_BACKGROUND_LANES = 10, /* 2-CTA shape: expert tiles of at most 64 rows are run by a second, small pipeline
                                         of every CTA pair (its own stage ring, TMA lane, MMA lane and accumulator)
                                         beside the pair's long tiles, so that the short tiles' weights stream in behind
                                         tensor-bound work.  1 (default): for batches of at least 4096 tokens of one
                                         model; 2: every batch of the 2-CTA shape; 0: never (one pipeline runs all tiles
                                         in turn).  Results are bit-identical. */
       MOE_OPT_ROUTE_LANES = 8 /* 2 (default): the tensor-core router issues its MMAs from two warps, even and odd K
                                  stages into two accumulators that the epilogue adds; 1: one warp, one accumulator
                                  (another summation order over K: logits differ in the last bits) */,
       MOE_OPT_FUSED_DISPATCH = 11 /* moe_layer_forward and the calls built on it, batches of at most 128 tokens of one
                                      model with the tensor-core router: 1: the router's one CTA goes on to batch the
                                      routed rows per expert block (Sec. 3, Sec. 4.1) and to lay out the experts' work,
                                      in the same launch; 0 (default): the dispatch is a launch of its own, as in
                                      moe_dispatch.  Results are bit-identical.  One launch fewer, but measured about
                                      1 % slower per step at 32 tokens: the dispatch kernel of its own is already
                                      resident and waiting when the router ends (programmatic dependent launch), and
                                      it keeps its tables in L1, which the router's CTA has given up for its stage
                                      ring. */,
       MOE_OPT_HEAD_UNITS = 12 /* moe_layer_forward and the calls built on it, batches of at most 64 tokens of one model
                                  with a shared expert: 1 (default): the gate/up launch works through the shared
                                  expert's units (tokens and static weights only) before it waits for the router and
                                  the dispatch of the same pass, so those weights stream in while the routing is being
                                  worked out; 0: it waits first.  Results are bit-identical. */ };

typedef struct {
    int32_t hidden;        /* H */
    int32_t n_experts;     /* E: routed experts per tenant model */
    int32_t inter;         /* I: intermediate size of one routed expert */
    int32_t top_k;         /* k */
    int32_t shared_inter;  /* I_s: intermediate size of the shared expert, 0 = none */
    int32_t n_models;      /* M: tenant models whose experts live in the pool */
    int32_t n_tenants;     /* tenant ids are 0 .. n_tenants-1 */
    int32_t n_slots;       /* S: routed-expert slots in the pool of each layer (>= 1) */
    int32_t max_tokens;    /* largest T any call will pass */
    int32_t n_layers;      /* L: 1 for a single layer */
    float   rms_eps;       /* epsilon of the RMSNorm in moe_stack_forward */
} moe_config;

/* Creates a context on the current device and allocates its workspace
 * (O(max_tokens * top_k * (2*H + I)) bytes).  cfg is a host pointer. */
int moe_create(const moe_config* cfg, moe_ctx** out);
int moe_destroy(moe_ctx* ctx);

/*
 * Registers the routed-expert pool of one layer (Sec. 4.1: experts are
 * extracted from each MoE layer and packaged by layer and expert id).
 *   w_gate, w_up : bf16 [S, I, H]    w_down : bf16 [S, H, I]
 * Slot s holds one SwiGLU expert: y = W_down . (silu(W_gate . x) * (W_up . x)).
 * The buffers are used in place.  16-byte aligned.  Where the tcgen05 kernels serve the
 * shape (hidden % 256 == 0), w_gate and w_up must be two distinct arrays whose addresses
 * differ by less than 2^40 bytes (one TMA descriptor walks both, with their distance as a
 * stride); otherwise MOE_ERR_UNSUPPORTED.  Two allocations of one process always qualify.
 */
int moe_set_expert_pool(moe_ctx* ctx, int layer, const void* w_gate, const void* w_up, const void* w_down);

/*
 * Registers the non-pooled weights of tenant model `model` in layer `layer`:
 *   router_w      bf16 [E, H]          gating network (Sec. 2.1)
 *   router_bias   f32  [E] or NULL     added to the router logits
 *   shared_gate_w bf16 [H] or NULL     sigmoid scalar gate of the shared expert
 *   ws_gate/ws_up bf16 [I_s, H], ws_down bf16 [H, I_s], or all NULL if I_s = 0
 *                                      (Sec. 5: the always-active shared experts)
 *   rms_w         bf16 [H] or NULL     RMSNorm scale, needed by moe_stack_forward only
 * Used in place; every pointer 16-byte aligned.  ws_gate and ws_up obey the same distance
 * rule as w_gate and w_up of moe_set_expert_pool (MOE_ERR_UNSUPPORTED otherwise).
 * Range: the shared expert's SwiGLU activations are kept in fp16 between its two
 * projections (its 4x longer contraction needs the finer mantissa); an activation
 * beyond +-65504 saturates there.  With weights and inputs of ordinary scale
 * (|activation| of a few units) that range is never approached.
 */
int moe_set_model_weights(moe_ctx* ctx, int layer, int model, const void* router_w, const float* router_bias,
                          const void* shared_gate_w, const void* ws_gate, const void* ws_up, const void* ws_down,
                          const void* rms_w);

/* Expert (m, e) lives in pool slot slot[m*E + e] (host pointer, M*E entries, each in
 * [0, S)).  The default is the identity m*E + e.  Copied; synchronises the device. */
int moe_set_slot_table(moe_ctx* ctx, const int32_t* slot);

/* Tenant u runs model model_of_tenant[u] (host pointer, n_tenants entries in [0, M)).
 * Default: u % M.  Copied; synchronises the device. */
int moe_set_tenant_models(moe_ctx* ctx, const int32_t* model_of_tenant);

/*
 * Load-aware formation of expert blocks (Sec. 5, on expert granularity: blocks that follow expert popularity are the
 * paper's outlook; the rule here is greedy).  For every model the E experts are put into B = ceil(E/G) blocks of at
 * most G experts so that the blocks' loads are even: experts in order of (load descending, id ascending), each into
 * the block with the smallest load so far among those with fewer than G experts (ties: lowest block id).
 * Host function, no GPU work: load is a host array [M, E] (for instance the per-expert row counts of earlier
 * batches, summed from tenant_expert_count), block_of_expert a host array [M, E] that receives ids in [0, B).
 */
int moe_form_blocks(const int64_t* load, int n_models, int n_experts, int G, int32_t* block_of_expert);

/*
 * Makes the context use blocks given by a table instead of blocks of G consecutive experts: block_of_expert is a host
 * array [M, E] of ids in [0, n_blocks) (copied; synchronises the device); NULL restores the ranges.  While a table is
 * set the G argument of the calls is only validated; a block is a set of experts, so group_off (M*n_blocks + 1
 * entries) holds the running sum of the rows the blocks receive, in block order, and the invocation statistics count
 * the table's blocks.  The permutation and every output bit stay the same (Sec. 3: block size and composition do not
 * affect routing or results); the table orders the expert work and defines what one invocation carries.
 */
int moe_set_block_table(moe_ctx* ctx, const int32_t* block_of_expert, int n_blocks);

int moe_set_option(moe_ctx* ctx, int option, int value);

/*
 * Gating (Sec. 2.1; Sec. 3: gating modules of the orchestrator).
 * For token t of tenant u = tenant_id[t], model m = model_of_tenant[u]:
 *   z[e] = x[t] . router_w[m][e] + bias[m][e]   (bf16 inputs, fp32 accumulation)
 *   p = softmax(z) in fp32; the k experts of largest p, ordered by (p descending,
 *   expert id ascending); weights are the raw probabilities (no renormalisation).
 *   shared_gate[t] = sigmoid(x[t] . shared_gate_w[m])
 *   tie_flag[t] = 1 if two neighbouring ranks among ranks 1..k+1 differ by less
 *   than 1e-5 relative (the order is then not decidable in fp32).
 * x bf16 [T,H]; tenant_id int32 [T]; topk_idx int32 [T,k]; topk_w f32 [T,k];
 * shared_gate f32 [T] or NULL; tie_flag u8 [T] or NULL.
 */
int moe_route(moe_ctx* ctx, int layer, const void* x, const int32_t* tenant_id, int T,
              int32_t* topk_idx, float* topk_w, float* shared_gate, uint8_t* tie_flag, void* stream);

/*
 * Micro-batched routing requests (Sec. 3; Sec. 4.1: all tokens routed to the same
 * expert block are consolidated into one batched invocation).
 * Row (t, j) has flat id t*k + j.  Rows are sorted by (model, expert, tenant, token):
 *   perm[r'] = flat id placed at position r';  inv_perm = its inverse      int32 [T*k]
 *   tenant_expert_count[u*E + e] = rows of tenant u routed to expert e    int32 [n_tenants*E]
 *   expert_off[m*E + e] = first position of expert (m,e); last entry T*k  int32 [M*E+1]
 *   group_off[m*B + b] = first position of block b = experts [b*G, min((b+1)*G, E))
 *                        of model m, B = ceil(E/G); last entry T*k        int32 [M*B+1]
 *   x_perm[r'] = x[perm[r'] / k]                                          bf16 [T*k, H] or NULL
 * perm does not depend on G (Sec. 3: block size does not affect routing correctness).
 * Any output pointer except perm/inv_perm/expert_off may be NULL.
 */
int moe_dispatch(moe_ctx* ctx, const void* x, const int32_t* topk_idx, const int32_t* tenant_id, int T, int G,
                 int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count, int32_t* expert_off,
                 int32_t* group_off, void* x_perm, void* stream);

/*
 * Expert execution (Sec. 3: an expert block keeps no state and computes only on the
 * tokens sent to it).  Only experts that received rows are touched.
 *   y_perm[r'] = FFN_{slot(m,e)}(x_perm[r'])    for r' in expert (m,e)'s segment   f32 [T*k, H]
 *   y_shared[t] = FFN_shared,m(x[t])  (ungated)                                    f32 [T, H] or NULL
 * (bf16 operands, fp32 accumulation; the SwiGLU activations are rounded to bf16 for the
 * routed experts and to fp16 for the shared expert before the down projection; the
 * results stay in fp32 so that the aggregation rounds only once)
 * G orders the work by expert block; results are bit-identical for every G.
 * x bf16 [T,H] and tenant_id are needed only when y_shared is requested.  perm (the
 * output of moe_dispatch) may be NULL; with x and perm given and at most 128 tokens of a
 * single model, the routed experts read the tokens in place instead of x_perm (same
 * results).
 */
int moe_experts(moe_ctx* ctx, int layer, const void* x, const void* x_perm, const int32_t* perm,
                const int32_t* expert_off, const int32_t* tenant_id, int T, int G, float* y_perm, float* y_shared,
                void* stream);

/*
 * Aggregation (Sec. 3, Sec. 4.2):
 *   out[t] = sum_{j=0..k-1} topk_w[t,j] * y_perm[inv_perm[t*k+j]] + shared_gate[t] * y_shared[t]
 * accumulated in fp32 in that fixed order, rounded once to bf16.  y_perm f32 [T*k,H],
 * y_shared f32 [T,H], out bf16 [T,H].
 * y_shared / shared_gate may both be NULL.
 */
int moe_combine(moe_ctx* ctx, const float* y_perm, const int32_t* inv_perm, const float* topk_w,
                const float* y_shared, const float* shared_gate, int T, void* out, void* stream);

/*
 * moe_dispatch for callers that must not allocate device memory (the paper has no
 * counterpart; this is a convenience of this library).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a host application
 * whose device memory pool is fixed at start-up, on a latency-critical path that cannot
 * afford cudaMalloc's implicit synchronisation, or in a process that already spent its
 * memory budget.  Such a caller cannot use moe_create either (it allocates the workspace),
 * so this call takes no context: the shapes and the tenant -> model table are arguments, and
 * the scratch the dispatch kernels need lives in a fixed array of
 * MOE_DISPATCH_NOALLOC_MAX_WORDS 32-bit words (1 MiB) inside the library, held by every GPU
 * that loads the library until the process exits.  The call itself and everything it
 * launches call no cudaMalloc, cudaFree or allocating library routine.
 *
 * Inputs and outputs are those of moe_dispatch (device pointers, same layouts and meaning,
 * without x / x_perm): topk_idx int32 [T,k], tenant_id int32 [T], model_of_tenant int32
 * [n_tenants] (DEVICE; an entry outside [0, M) counts as model 0), perm / inv_perm int32 [T*k], tenant_expert_count int32
 * [n_tenants*E] or NULL, expert_off int32 [M*E+1], group_off int32 [M*ceil(E/G)+1] or NULL.
 * status_out, if not NULL, is a device int32 that receives the MOE_DEV_* bits of this call
 * (it is cleared first, also when T = 0 and nothing else is launched).
 *
 * Limit: 10 + 2*n_tenants + 2*M + (ceil(T*k/256) + 1) * E*n_tenants words must fit in the
 * array; larger problems return MOE_ERR_UNSUPPORTED and launch nothing.
 * The first call on each device looks up the array's device address; make that first call
 * before any stream capture.  All calls on a device share the array and it keeps the last
 * call's contents (what must start at zero is cleared by the call itself): two calls that
 * overlap on the GPU -- different streams, or different host threads -- race on it.
 */
#define MOE_DISPATCH_NOALLOC_MAX_WORDS (1 << 18)
int moe_dispatch_noalloc(const int32_t* topk_idx, const int32_t* tenant_id, const int32_t* model_of_tenant,
                         int T, int k, int E, int M, int n_tenants, int G, int32_t* perm, int32_t* inv_perm,
                         int32_t* tenant_expert_count, int32_t* expert_off, int32_t* group_off,
                         int32_t* status_out, void* stream);

/* route -> dispatch -> experts -> combine on the context's workspace; bit-identical to
 * the four calls above.  out bf16 [T,H]. */
int moe_layer_forward(moe_ctx* ctx, int layer, const void* x, const int32_t* tenant_id, int T, int G,
                      void* out, void* stream);

/*
 * On-demand residency of the routed experts: the device-side analogue of functions that scale to zero (abstract;
 * Sec. 3: rarely used experts need not hold resources while idle).  All M*E experts of the layer are parked in HOST
 * memory (host_gate / host_up bf16 [M*E, I, H], host_down bf16 [M*E, H, I], indexed by m*E + e; pinned memory makes
 * the copies asynchronous); the pool on the device (pool_* = DEVICE arrays of n_slots slots, registered as by
 * moe_set_expert_pool) is a cache of the experts in use, and the slot table is managed by the library.  One layer per
 * context (MOE_ERR_UNSUPPORTED otherwise).
 */
int moe_residency_enable(moe_ctx* ctx, int layer, const void* host_gate, const void* host_up, const void* host_down,
                         void* pool_gate, void* pool_up, void* pool_down);

/*
 * moe_layer_forward with on-demand residency: runs the gate, reads the set of experts the batch routes to back to the
 * host (this call synchronises `stream` once, after the gate), copies every needed expert that is parked into a slot
 * -- a free one (lowest index) or else the one used longest ago among those this batch does not need (ties: lowest
 * index; experts are taken in ascending id) -- and runs dispatch, experts and combine on the routing already made.
 * Results are bit-identical to a context that keeps every expert resident.  More active experts than slots:
 * MOE_ERR_UNSUPPORTED.  stats_host (host, 4 ints, or NULL): active experts, resident hits, experts loaded, experts
 * evicted by this call.
 */
int moe_layer_forward_paged(moe_ctx* ctx, int layer, const void* x, const int32_t* tenant_id, int T, int G, void* out,
                            int32_t* stats_host, void* stream);

/* Same, with HOST buffers: copies x and tenant_id to the device, runs the layer,
 * copies out back and synchronises the stream.  For best speed pass pinned memory. */
int moe_layer_forward_host(moe_ctx* ctx, int layer, const void* x_host, const int32_t* tenant_id_host, int T, int G,
                           void* out_host, void* stream);

/*
 * The host-buffer call as a pipeline: submit enqueues the copy of x_host / tenant_id_host to the device (on a copy
 * stream of the context), the layer (on `stream`, after the copy) and the copy of the result to out_host (on a second
 * copy stream, after the layer), and returns a ticket without waiting; wait blocks until out_host of that ticket is
 * complete.  Two submissions may be in flight: the third submit first waits for the first one's outputs (its staging
 * buffers are reused).  The inputs of one call then travel while the previous call computes and the call before that
 * returns its outputs, so a stream of calls runs at the slowest of the three instead of their sum.  x_host,
 * tenant_id_host and out_host must be pinned and stay valid until the ticket has been waited for.  Results are those of
 * moe_layer_forward_host.
 */
int moe_layer_forward_host_submit(moe_ctx* ctx, int layer, const void* x_host, const int32_t* tenant_id_host, int T, int G,
                                  void* out_host, void* stream, int64_t* ticket);
int moe_layer_forward_host_wait(moe_ctx* ctx, int64_t ticket);

/* moe_layer_forward with a CUDA event recorded on `stream` after every stage; synchronises the
 * stream and writes the stage durations in milliseconds to stage_ms_host (host, 6 floats):
 * route, dispatch, plan, experts gate/up, experts down, combine. */
int moe_layer_forward_timed(moe_ctx* ctx, int layer, const void* x, const int32_t* tenant_id, int T, int G,
                            void* out, float* stage_ms_host, void* stream);

/*
 * n_layers blocks of: xn = bf16(RMSNorm(x) * rms_w);  o = layer(xn);  x = bf16(x + o).
 * x_inout bf16 [T,H] is updated in place.  dbg_layer_inputs, if not NULL, receives the
 * xn of every block, and dbg_layer_outputs, if not NULL, the residual stream x after every
 * block: bf16 [L, T, H] each.
 */
int moe_stack_forward(moe_ctx* ctx, void* x_inout, const int32_t* tenant_id, int T, int G,
                      void* dbg_layer_inputs, void* dbg_layer_outputs, void* stream);

/* Device pointers into the workspace holding the routing results of the last
 * moe_layer_forward (valid until the next call on this context). */
int moe_get_workspace(moe_ctx* ctx, int32_t** topk_idx, float** topk_w, float** shared_gate, uint8_t** tie_flag,
                      int32_t** perm, int32_t** inv_perm, int32_t** expert_off, int32_t** group_off);

/* Synchronises the device, returns the device status word in *status_host and clears it.
 * Also reports, if not NULL, stats_host[0] = invocations of the last dispatch (shared
 * orchestrator: non-empty expert blocks; private orchestrators: (tenant, block) pairs with
 * rows -- see MOE_OPT_DISPATCH_MODE) and stats_host[1] = its active routed experts. */
int moe_last_status(moe_ctx* ctx, int32_t* status_host, int32_t* stats_host);

/* Synchronises the device and reports how the last moe_experts / moe_layer_forward call on this context cut the
 * expert work (Sec. 4.1: requests are batched per block; Sec. 4.2: per tenant too under private orchestrators):
 * plan_host[0] = tiles of routed rows, plan_host[1] = tiles of shared-expert tokens, plan_host[2] = most rows a
 * tile holds at batch size T.  plan_host is a host pointer to 3 ints. */
int moe_last_plan(moe_ctx* ctx, int T, int32_t* plan_host);

/* Number of kernels this library has launched on this context since creation. */
int64_t moe_launch_count(moe_ctx* ctx);

const char* moe_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* FAASMOE_H */
