/*
 * moe_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of the multi-tenant Mixture-of-Experts
 * layer that FaaSMoE serves: gating network + top-k selection (paper Sec. 2.1),
 * grouping of the routed tokens into one request per expert block (Sec. 3,
 * Sec. 4.1), stateless expert execution on the assigned tokens (Sec. 3), and
 * aggregation of the expert outputs per token (Sec. 3, Sec. 4.2).
 *
 * Nothing here is tuned.  Every function is the textbook definition written
 * as loops over tokens, experts and features; inputs are the exact values of
 * the bf16 operands widened to double and nothing is rounded on the way.
 * OpenMP only spreads independent tokens / rows over host cores.
 *
 * This file shares no code with the CUDA library.  Only tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.
 *
 * The paper prints no equations; the numeric details it leaves open (SwiGLU
 * experts, softmax over all experts without renormalisation, sigmoid-gated
 * shared expert, tie-breaking, segment order) are the readings listed in the
 * design notes of this repository.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> double: a bf16 is the upper half of an IEEE binary32. */
static inline double bf16_to_f64(uint16_t v)
{
    uint32_t bits = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static inline double silu(double a) { return a / (1.0 + exp(-a)); }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* dot product of two bf16 vectors, index ascending, fp64 */
static double dot_bf16(const uint16_t* a, const uint16_t* b, int n)
{
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += bf16_to_f64(a[i]) * bf16_to_f64(b[i]);
    return s;
}

/*
 * Gating network (Sec. 2.1: a gate picks the k best experts of every token;
 * Sec. 3: the gating modules live in the orchestrator).
 *
 *   z[t,e] = sum_h x[t,h] * W_r[m][e,h] + b[m][e]      m = model_of_tenant[tenant_id[t]]
 *   p[t,:] = softmax_e(z[t,:])
 *   experts ordered by (p descending, e ascending); the first k are selected,
 *   their weights are the raw probabilities (no renormalisation).
 *   shared_gate[t] = sigmoid( w_sg[m] . x[t] )           (if w_sg given)
 *   tie_flag[t] = 1 if two neighbouring ranks among ranks 1..k+1 are closer
 *                 than 1e-5 relative (the selection or its order is then not
 *                 decidable in fp32).
 *
 * x [T,H] bf16; router_w [M,E,H] bf16; router_bias [M,E] f32 or NULL;
 * shared_gate_w [M,H] bf16 or NULL.  Outputs: probs [T,E] (or NULL),
 * topk_idx [T,k], topk_w [T,k], shared_gate [T] (or NULL), tie_flag [T] (or NULL).
 * Returns 0, or -1 on an out-of-range tenant id.
 */
int oracle_route(const uint16_t* x, const int32_t* tenant_id, int T, int H, int E, int k,
                 int n_models, int n_tenants, const int32_t* model_of_tenant,
                 const uint16_t* router_w, const float* router_bias,
                 const uint16_t* shared_gate_w,
                 double* probs, int32_t* topk_idx, double* topk_w,
                 double* shared_gate, uint8_t* tie_flag)
{
    int bad = 0;
    for (int t = 0; t < T; ++t) {
        if (tenant_id[t] < 0 || tenant_id[t] >= n_tenants) bad = 1;
        else if (model_of_tenant[tenant_id[t]] < 0 || model_of_tenant[tenant_id[t]] >= n_models) bad = 1;
    }
    if (bad) return -1;

#pragma omp parallel for schedule(dynamic, 4)
    for (int t = 0; t < T; ++t) {
        const int m = model_of_tenant[tenant_id[t]];
        const uint16_t* xt = x + (size_t)t * H;
        double* z = (double*)malloc(sizeof(double) * (size_t)E);
        double* p = (double*)malloc(sizeof(double) * (size_t)E);
        int* order = (int*)malloc(sizeof(int) * (size_t)E);

        for (int e = 0; e < E; ++e) {
            z[e] = dot_bf16(xt, router_w + ((size_t)m * E + e) * H, H);
            if (router_bias) z[e] += (double)router_bias[(size_t)m * E + e];
        }
        double zmax = z[0];
        for (int e = 1; e < E; ++e) if (z[e] > zmax) zmax = z[e];
        double den = 0.0;
        for (int e = 0; e < E; ++e) { p[e] = exp(z[e] - zmax); den += p[e]; }
        for (int e = 0; e < E; ++e) p[e] /= den;
        if (probs) for (int e = 0; e < E; ++e) probs[(size_t)t * E + e] = p[e];

        /* insertion sort of expert ids by (p desc, id asc): stable, so equal
           probabilities keep ascending id order */
        for (int e = 0; e < E; ++e) order[e] = e;
        for (int i = 1; i < E; ++i) {
            int cur = order[i];
            int j = i - 1;
            while (j >= 0 && p[order[j]] < p[cur]) { order[j + 1] = order[j]; --j; }
            order[j + 1] = cur;
        }
        for (int j = 0; j < k; ++j) {
            topk_idx[(size_t)t * k + j] = order[j];
            topk_w[(size_t)t * k + j] = p[order[j]];
        }
        if (tie_flag) {
            uint8_t f = 0;
            int last = (k < E) ? k : E - 1;      /* compare ranks (i, i+1), i = 0..last-1 (0-based) */
            for (int i = 0; i < last; ++i) {
                double hi = p[order[i]], lo = p[order[i + 1]];
                if (hi - lo < 1e-5 * hi) f = 1;
            }
            tie_flag[t] = f;
        }
        if (shared_gate) {
            double a = shared_gate_w ? dot_bf16(xt, shared_gate_w + (size_t)m * H, H) : 0.0;
            shared_gate[t] = 1.0 / (1.0 + exp(-a));
        }
        free(z); free(p); free(order);
    }
    return 0;
}

/*
 * Routing requests, batched per expert block (Sec. 3: the orchestrator groups
 * the routed tokens into one request per block; Sec. 4.1: whatever goes to the
 * same block travels in one invocation; blocks are packaged by layer and
 * expert id, G experts per block).
 *
 * A routed row is (t, j) with flat id t*k + j.  Rows are ordered by the key
 *   (model, expert, tenant, token)
 * so that every expert's rows, and inside them every tenant's rows, are
 * contiguous and every block of G consecutive experts of one model is one
 * contiguous range of rows.
 *
 * Outputs: perm [T*k] (perm[r'] = flat row id placed at position r'),
 * inv_perm [T*k], tenant_expert_count [n_tenants,E], expert_off [M*E+1],
 * group_off [M*B+1] with B = ceil(E/G), *n_invocations = number of non-empty
 * blocks.  Returns 0, -1 on bad tenant/expert ids, -2 on bad G.
 */
int oracle_dispatch(const int32_t* topk_idx, const int32_t* tenant_id, int T, int E, int k,
                    int n_models, int n_tenants, const int32_t* model_of_tenant, int G,
                    int32_t* perm, int32_t* inv_perm, int32_t* tenant_expert_count,
                    int32_t* expert_off, int32_t* group_off, int32_t* n_invocations)
{
    if (G < 1 || G > E) return -2;
    const int R = T * k;
    const int B = (E + G - 1) / G;
    for (int t = 0; t < T; ++t) {
        if (tenant_id[t] < 0 || tenant_id[t] >= n_tenants) return -1;
        int m = model_of_tenant[tenant_id[t]];
        if (m < 0 || m >= n_models) return -1;
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            if (e < 0 || e >= E) return -1;
        }
    }
    memset(tenant_expert_count, 0, sizeof(int32_t) * (size_t)n_tenants * E);
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j)
            tenant_expert_count[(size_t)tenant_id[t] * E + topk_idx[(size_t)t * k + j]] += 1;

    /* selection by exhaustive walk in key order: for each (model, expert,
       tenant) in ascending order, append that bin's rows in token order */
    int pos = 0;
    for (int m = 0; m < n_models; ++m) {
        for (int e = 0; e < E; ++e) {
            expert_off[(size_t)m * E + e] = pos;
            for (int u = 0; u < n_tenants; ++u) {
                if (model_of_tenant[u] != m) continue;
                for (int t = 0; t < T; ++t) {
                    if (tenant_id[t] != u) continue;
                    for (int j = 0; j < k; ++j) {
                        if (topk_idx[(size_t)t * k + j] == e) {
                            perm[pos] = t * k + j;
                            inv_perm[t * k + j] = pos;
                            ++pos;
                        }
                    }
                }
            }
        }
    }
    expert_off[(size_t)n_models * E] = pos;
    if (pos != R) return -1;   /* a tenant mapped to no model in range */

    int ninv = 0;
    for (int m = 0; m < n_models; ++m) {
        for (int b = 0; b < B; ++b) {
            int e0 = b * G;
            int e1 = e0 + G; if (e1 > E) e1 = E;
            group_off[(size_t)m * B + b] = expert_off[(size_t)m * E + e0];
            if (expert_off[(size_t)m * E + e1] > expert_off[(size_t)m * E + e0]) ++ninv;
        }
    }
    group_off[(size_t)n_models * B] = R;
    if (n_invocations) *n_invocations = ninv;
    return 0;
}

/*
 * Load-aware formation of expert blocks (Sec. 5, on expert granularity: the
 * paper leaves blocks that take expert popularity into account as future
 * work; the reading taken here is the greedy rule below).
 *
 * For every model, its E experts are put into B = ceil(E/G) blocks of at most
 * G experts each so that the blocks' loads are even: experts are taken in the
 * order (load descending, expert id ascending) and each goes to the block that
 * has the smallest load so far among the blocks with fewer than G experts
 * (ties: the lowest block id).
 *
 * load [M,E] (rows routed to every expert, any non-negative weights);
 * block_of_expert [M,E] receives block ids in [0, B).  Returns 0, -2 on bad G.
 */
int oracle_form_blocks(const int64_t* load, int n_models, int E, int G, int32_t* block_of_expert)
{
    if (G < 1 || G > E) return -2;
    const int B = (E + G - 1) / G;
    int* order = (int*)malloc(sizeof(int) * (size_t)E);
    int64_t* bload = (int64_t*)malloc(sizeof(int64_t) * (size_t)B);
    int* bsize = (int*)malloc(sizeof(int) * (size_t)B);
    for (int m = 0; m < n_models; ++m) {
        const int64_t* l = load + (size_t)m * E;
        for (int e = 0; e < E; ++e) order[e] = e;
        /* insertion sort by (load descending, id ascending) */
        for (int i = 1; i < E; ++i) {
            const int v = order[i];
            int j = i - 1;
            while (j >= 0 && (l[order[j]] < l[v] || (l[order[j]] == l[v] && order[j] > v))) { order[j + 1] = order[j]; --j; }
            order[j + 1] = v;
        }
        for (int b = 0; b < B; ++b) { bload[b] = 0; bsize[b] = 0; }
        for (int i = 0; i < E; ++i) {
            const int e = order[i];
            int best = -1;
            for (int b = 0; b < B; ++b)
                if (bsize[b] < G && (best < 0 || bload[b] < bload[best])) best = b;
            block_of_expert[(size_t)m * E + e] = best;
            bload[best] += l[e];
            bsize[best] += 1;
        }
    }
    free(order); free(bload); free(bsize);
    return 0;
}

/*
 * Invocation accounting for blocks given by a table (block_of_expert [M,E],
 * ids in [0, n_blocks)) instead of ranges of G consecutive experts; same
 * meaning of mode and of the outputs as oracle_invocations below.  block_rows
 * [M, n_blocks] (or NULL) receives the rows every block gets.
 */
int oracle_invocations_table(const int32_t* topk_idx, const int32_t* tenant_id, int T, int E, int k,
                             int n_models, int n_tenants, const int32_t* model_of_tenant,
                             const int32_t* block_of_expert, int n_blocks, int mode,
                             int32_t* n_invocations, int32_t* tenant_invocations, int32_t* token_fanout,
                             int32_t* block_rows)
{
    if (mode < 0 || mode > 1 || n_blocks < 1) return -2;
    for (int i = 0; i < n_models * E; ++i) if (block_of_expert[i] < 0 || block_of_expert[i] >= n_blocks) return -1;
    /* reached[u][b]: tenant u has a row in block b of its model */
    unsigned char* reached = (unsigned char*)calloc((size_t)n_tenants * n_blocks, 1);
    unsigned char* any = (unsigned char*)calloc((size_t)n_models * n_blocks, 1);
    if (block_rows) memset(block_rows, 0, sizeof(int32_t) * (size_t)n_models * n_blocks);
    for (int t = 0; t < T; ++t) {
        const int u = tenant_id[t];
        if (u < 0 || u >= n_tenants || model_of_tenant[u] < 0 || model_of_tenant[u] >= n_models) { free(reached); free(any); return -1; }
        const int m = model_of_tenant[u];
        int fan = 0;
        for (int j = 0; j < k; ++j) {
            const int e = topk_idx[(size_t)t * k + j];
            if (e < 0 || e >= E) { free(reached); free(any); return -1; }
            const int b = block_of_expert[(size_t)m * E + e];
            reached[(size_t)u * n_blocks + b] = 1;
            any[(size_t)m * n_blocks + b] = 1;
            if (block_rows) block_rows[(size_t)m * n_blocks + b] += 1;
            int seen = 0;
            for (int j2 = 0; j2 < j; ++j2)
                if (block_of_expert[(size_t)m * E + topk_idx[(size_t)t * k + j2]] == b) seen = 1;
            if (!seen) ++fan;
        }
        if (token_fanout) token_fanout[t] = fan;
    }
    int ninv = 0;
    for (int u = 0; u < n_tenants; ++u) {
        int c = 0;
        for (int b = 0; b < n_blocks; ++b) c += reached[(size_t)u * n_blocks + b];
        if (tenant_invocations) tenant_invocations[u] = c;
        if (mode == 1) ninv += c;
    }
    if (mode == 0)
        for (int i = 0; i < n_models * n_blocks; ++i) ninv += any[i];
    free(reached); free(any);
    if (n_invocations) *n_invocations = ninv;
    return 0;
}

/*
 * Invocation accounting of the two orchestrator placements (Sec. 4.2,
 * deployment strategies FaaSMoE-Shared and FaaSMoE-Private; Sec. 4.3.1 on
 * batching across tenants and fan-out; Sec. 5 on orchestrator placement).
 *
 *   mode 0, shared orchestrator: one orchestrator serves every tenant, so all
 *     rows that reach a block travel in ONE invocation whoever owns them:
 *     invocations = blocks (m, b) that received at least one row.
 *   mode 1, private orchestrators: every tenant has an orchestrator of its own
 *     that batches only its own tokens: invocations = pairs (tenant u, block b
 *     of u's model) with at least one row of u.
 *
 * Outputs (any may be NULL):
 *   *n_invocations        as above
 *   tenant_invocations[u] blocks that rows of tenant u reach (private: the
 *                         invocations u's orchestrator issues, they sum to
 *                         *n_invocations; shared: how many of the shared
 *                         invocations carry rows of u)
 *   token_fanout[t]       distinct blocks among the k experts of token t (the
 *                         invocations one token takes part in; same in both modes)
 *   *n_row_batches        row batches when the rows that ONE invocation sends to
 *                         ONE expert are cut into pieces of at most batch_rows
 *                         rows: shared sum over (m,e) of ceil(cnt/batch_rows),
 *                         private sum over (u,e)
 * Returns 0, -1 on bad ids, -2 on bad G / mode / batch_rows.
 */
int oracle_invocations(const int32_t* topk_idx, const int32_t* tenant_id, int T, int E, int k,
                       int n_models, int n_tenants, const int32_t* model_of_tenant, int G, int mode,
                       int batch_rows, int32_t* n_invocations, int32_t* tenant_invocations,
                       int32_t* token_fanout, int32_t* n_row_batches)
{
    if (G < 1 || G > E || mode < 0 || mode > 1 || batch_rows < 1) return -2;
    const int B = (E + G - 1) / G;
    /* rows[u][e]: rows of tenant u routed to expert e */
    int32_t* rows = (int32_t*)calloc((size_t)n_tenants * E, sizeof(int32_t));
    for (int t = 0; t < T; ++t) {
        const int u = tenant_id[t];
        if (u < 0 || u >= n_tenants || model_of_tenant[u] < 0 || model_of_tenant[u] >= n_models) { free(rows); return -1; }
        int fan = 0;
        for (int j = 0; j < k; ++j) {
            const int e = topk_idx[(size_t)t * k + j];
            if (e < 0 || e >= E) { free(rows); return -1; }
            rows[(size_t)u * E + e] += 1;
            int seen = 0;                       /* was this block already counted for the token? */
            for (int j2 = 0; j2 < j; ++j2) if (topk_idx[(size_t)t * k + j2] / G == e / G) seen = 1;
            if (!seen) ++fan;
        }
        if (token_fanout) token_fanout[t] = fan;
    }
    int ninv = 0, nbatch = 0;
    if (tenant_invocations) memset(tenant_invocations, 0, sizeof(int32_t) * (size_t)n_tenants);
    /* blocks reached per tenant */
    for (int u = 0; u < n_tenants; ++u) {
        for (int b = 0; b < B; ++b) {
            int any = 0;
            for (int e = b * G; e < E && e < (b + 1) * G; ++e) if (rows[(size_t)u * E + e] > 0) any = 1;
            if (any) {
                if (tenant_invocations) tenant_invocations[u] += 1;
                if (mode == 1) ++ninv;
            }
        }
        if (mode == 1)
            for (int e = 0; e < E; ++e) nbatch += (rows[(size_t)u * E + e] + batch_rows - 1) / batch_rows;
    }
    if (mode == 0) {
        for (int m = 0; m < n_models; ++m) {
            for (int b = 0; b < B; ++b) {
                int any = 0;
                for (int e = b * G; e < E && e < (b + 1) * G; ++e) {
                    int cnt = 0;
                    for (int u = 0; u < n_tenants; ++u) if (model_of_tenant[u] == m) cnt += rows[(size_t)u * E + e];
                    if (cnt > 0) any = 1;
                    nbatch += (cnt + batch_rows - 1) / batch_rows;
                }
                if (any) ++ninv;
            }
        }
    }
    free(rows);
    if (n_invocations) *n_invocations = ninv;
    if (n_row_batches) *n_row_batches = nbatch;
    return 0;
}

/*
 * One SwiGLU expert on one token (Sec. 3: an expert block keeps no state and
 * computes on the tokens it was sent; Sec. 5: experts are small MLPs):
 *   y = W_d . ( silu(W_g . x) * (W_u . x) )
 * W_g, W_u [I,H]; W_d [H,I]; all bf16 row-major.  scratch holds I doubles.
 */
static void swiglu_ffn(const uint16_t* x, int H, int I,
                       const uint16_t* wg, const uint16_t* wu, const uint16_t* wd,
                       double* scratch, double* y)
{
    for (int i = 0; i < I; ++i) {
        double g = dot_bf16(x, wg + (size_t)i * H, H);
        double u = dot_bf16(x, wu + (size_t)i * H, H);
        scratch[i] = silu(g) * u;
    }
    for (int h = 0; h < H; ++h) {
        const uint16_t* row = wd + (size_t)h * I;
        double s = 0.0;
        for (int i = 0; i < I; ++i) s += bf16_to_f64(row[i]) * scratch[i];
        y[h] = s;
    }
}

/*
 * Expert execution over the routed rows, in segment order (Sec. 3, Sec. 4.1).
 * Only the experts that received rows are touched.
 *
 * pool_gate/pool_up [S,I,H], pool_down [S,H,I]: the shared expert pool;
 * slot_table [M*E]: expert (m,e) lives in pool slot slot_table[m*E+e]
 * (Sec. 4.1: experts are extracted and packaged by layer and expert id).
 * y_perm [T*k,H] double.  Returns 0 or -1 on a bad index.
 */
int oracle_experts(const uint16_t* x, const int32_t* tenant_id, const int32_t* topk_idx,
                   const int32_t* perm, int T, int H, int E, int I, int k,
                   int n_models, const int32_t* model_of_tenant,
                   const uint16_t* pool_gate, const uint16_t* pool_up, const uint16_t* pool_down,
                   int n_slots, const int32_t* slot_table, double* y_perm)
{
    const int R = T * k;
    int bad = 0;
#pragma omp parallel
    {
        double* scratch = (double*)malloc(sizeof(double) * (size_t)I);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < R; ++r) {
            int row = perm[r];
            if (row < 0 || row >= R) { bad = 1; continue; }
            int t = row / k;
            int e = topk_idx[row];
            int m = model_of_tenant[tenant_id[t]];
            if (e < 0 || e >= E || m < 0 || m >= n_models) { bad = 1; continue; }
            int s = slot_table[(size_t)m * E + e];
            if (s < 0 || s >= n_slots) { bad = 1; continue; }
            swiglu_ffn(x + (size_t)t * H, H, I,
                       pool_gate + (size_t)s * I * H, pool_up + (size_t)s * I * H,
                       pool_down + (size_t)s * H * I, scratch, y_perm + (size_t)r * H);
        }
        free(scratch);
    }
    return bad ? -1 : 0;
}

/*
 * The always-active shared expert of each model (Sec. 5: "60 experts and 4
 * shared experts per MoE layer"; the four are one SwiGLU of 4x the width).
 * ws_gate/ws_up [M,Is,H], ws_down [M,H,Is]; y_shared [T,H] double, ungated.
 */
int oracle_shared_expert(const uint16_t* x, const int32_t* tenant_id, int T, int H, int Is,
                         int n_models, const int32_t* model_of_tenant,
                         const uint16_t* ws_gate, const uint16_t* ws_up, const uint16_t* ws_down,
                         double* y_shared)
{
    int bad = 0;
#pragma omp parallel
    {
        double* scratch = (double*)malloc(sizeof(double) * (size_t)Is);
#pragma omp for schedule(dynamic, 1)
        for (int t = 0; t < T; ++t) {
            int m = model_of_tenant[tenant_id[t]];
            if (m < 0 || m >= n_models) { bad = 1; continue; }
            swiglu_ffn(x + (size_t)t * H, H, Is,
                       ws_gate + (size_t)m * Is * H, ws_up + (size_t)m * Is * H,
                       ws_down + (size_t)m * H * Is, scratch, y_shared + (size_t)t * H);
        }
        free(scratch);
    }
    return bad ? -1 : 0;
}

/*
 * Aggregation (Sec. 3: the orchestrator puts the expert outputs of a token together;
 * Sec. 4.2 lists it among the orchestrator's duties):
 *   out[t] = sum_{j=0..k-1} w[t,j] * y_perm[inv_perm[t*k+j]]  +  s[t] * y_shared[t]
 * y_shared / shared_gate may be NULL (no shared expert).  out [T,H] double.
 */
int oracle_combine(const double* y_perm, const int32_t* inv_perm, const double* topk_w,
                   const double* y_shared, const double* shared_gate,
                   int T, int H, int k, double* out)
{
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h) {
            double s = 0.0;
            for (int j = 0; j < k; ++j) {
                int r = inv_perm[(size_t)t * k + j];
                s += topk_w[(size_t)t * k + j] * y_perm[(size_t)r * H + h];
            }
            if (y_shared) s += shared_gate[t] * y_shared[(size_t)t * H + h];
            out[(size_t)t * H + h] = s;
        }
    }
    return 0;
}

/*
 * RMSNorm in front of a block of the stacked configuration:
 *   xn[t,h] = x[t,h] * (mean_h x[t,h]^2 + eps)^(-1/2) * g[h]       (fp64)
 * x [T,H] bf16, g [H] bf16, xn [T,H] double (the caller rounds to bf16).
 */
int oracle_rmsnorm(const uint16_t* x, const uint16_t* g, int T, int H, double eps, double* xn)
{
    for (int t = 0; t < T; ++t) {
        double ss = 0.0;
        for (int h = 0; h < H; ++h) {
            double v = bf16_to_f64(x[(size_t)t * H + h]);
            ss += v * v;
        }
        double r = 1.0 / sqrt(ss / (double)H + eps);
        for (int h = 0; h < H; ++h)
            xn[(size_t)t * H + h] = bf16_to_f64(x[(size_t)t * H + h]) * r * bf16_to_f64(g[h]);
    }
    return 0;
}

/*
 * Round doubles to bf16 (round-to-nearest, ties-to-even) in a single
 * rounding step.  Used between the blocks of the stacked configuration,
 * where the residual stream is stored in bf16.  Finite inputs only.
 */
void oracle_round_bf16(const double* v, size_t n, uint16_t* out)
{
    for (size_t i = 0; i < n; ++i) {
        double a = fabs(v[i]);
        float f = (float)a;                       /* within half a binary32 ulp of a */
        uint32_t bits;
        memcpy(&bits, &f, sizeof bits);
        uint32_t lo_bits = bits & 0xFFFF0000u;    /* bf16 neighbour at or below f */
        uint32_t hi_bits = lo_bits + 0x00010000u; /* next bf16 above */
        float lo_f, hi_f;
        memcpy(&lo_f, &lo_bits, sizeof lo_f);
        memcpy(&hi_f, &hi_bits, sizeof hi_f);
        double dl = a - (double)lo_f;             /* may be slightly negative: picks lo */
        double du = (double)hi_f - a;
        uint32_t pick;
        if (dl < du) pick = lo_bits;
        else if (du < dl) pick = hi_bits;
        else pick = (lo_bits & 0x00010000u) ? hi_bits : lo_bits;
        uint16_t r = (uint16_t)(pick >> 16);
        if (v[i] < 0.0 || (v[i] == 0.0 && signbit(v[i]))) r |= 0x8000u;
        out[i] = r;
    }
}
