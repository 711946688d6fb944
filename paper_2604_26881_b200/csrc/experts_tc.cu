// Tensor-core expert execution for sm_100a: one persistent, warp-specialised grouped GEMM
// (TMA -> shared memory -> tcgen05.mma -> TMEM -> registers) used twice per layer:
//   gate/up:  h[r, c]  = silu(W_g[c,:] . x[r,:]) * (W_u[c,:] . x[r,:])        (SwiGLU in the epilogue)
//   down:     y[r, c]  = W_d[c,:] . h[r,:]
// (paper Sec. 3: an expert block computes on the tokens assigned to it; only activated experts are
// touched.)
//
// Three shapes of the same kernel (all give bit-identical results: every output element is accumulated over K
// in the same order):
//   token-major (SWAP): one CTA per unit; the tokens of an expert tile (at most 128) are the M operand, one
//     TMEM lane per token, and 256 weight rows the N operand (128 or 64 for the narrow units of the plan).
//     For gate/up a 3-D TMA box over the two weight arrays interleaves gate and up rows, which land on
//     neighbouring TMEM columns of a token's lane: SwiGLU needs no cross-lane traffic.  This is the
//     weight-streaming shape of small batches: up to 64 tokens (decode), where the routed units also read
//     the tokens in place.  One MMA covers 256 weight rows, and an MMA costs its issuing lane about 100 cycles whatever
//     its width, so few tokens are bound by HBM, not by MMA issue.
//   pair (PAIR): a cluster of two CTAs works on one unit through tcgen05.mma.cta_group::2; the weight rows
//     are the M operand (128 per CTA), the tokens N: up to 512 per unit in two 256-column accumulators fed from
//     the same weight tile, each CTA loading half of the tokens; short units put two K slices into a stage.
//     Used for every batch above 64 tokens.
//   weight-major, one CTA (neither flag): 128 weight rows as M, at most 128 tokens as N; kept as the A/B
//     reference of the other two.
// Routed-expert units and shared-expert units ride in the same launch.
#include <cuda_fp16.h>

#include <algorithm>
#include <cstdio>
#include <cstring>

#include "internal.h"
#include "tc_ptx.cuh"

namespace faasmoe {

namespace {

using namespace tc;

constexpr int kMaxStages = 6;
constexpr int kBarBytesDecl = 512;
constexpr int kBK = 64;                        // K elements per stage = one 128-byte swizzle row
constexpr int kABytes = 128 * kBK * 2;         // 128 weight rows: 16 KB
constexpr int kBRows = 128;                    // token rows one CTA loads per accumulator and stage (pair: half of them)
constexpr int kBBytes = kBRows * kBK * 2;      // 16 KB
// Two pipeline geometries over the same 192 KB: 6 stages of (weights + one token tile), or 4 stages of
// (weights + two token tiles) when a unit may feed both accumulators from one weight tile ("wide" units).
constexpr int kRingBytes = kMaxStages * (kABytes + kBBytes);
constexpr int kWideStages = kRingBytes / (kABytes + 2 * kBBytes);
constexpr int kQueue = 4;                      // depth of the unit queue of the dynamic scheduler
// The background pipeline of the pair shape (see the kernel): a ring, a unit queue and an accumulator of its own.
constexpr int kBgStages = 4;
constexpr int kBgRows = kShortRows / 2;        // token rows one CTA of the pair loads per stage (at most)
constexpr int kBgStageBytes = kABytes + kBgRows * kBK * 2;      // 20 KB: 128 weight rows + 32 token rows
constexpr int kBgRingBytes = kBgStages * kBgStageBytes;         // 60 KB
constexpr int kBgQueue = 2;
constexpr int kBgAccRows = kAccRowsBg;         // token rows per accumulator of a wide tile when the background pipeline runs
constexpr int kBgStageBytesMain = kABytes + 2 * (kBgAccRows / 2) * kBK * 2;    // 44 KB: weights + two token tiles of 112 rows
constexpr int kBgMainStages = 3;               // (4 main + 2 background stages measured no better: the background lanes, bound
                                               // by the latency of their few stages in flight, then become the long pole)
// the two rings take 212 KB: with the background pipeline the epilogue writes its results straight to global memory
// and the 32 KB output staging area goes to the rings
constexpr int kBgRingsBytes = kBgMainStages * kBgStageBytesMain + kBgRingBytes;

static_assert(kBgStageBytesMain % 1024 == 0 && kBgStageBytes % 1024 == 0, "swizzled tiles need 1024-byte alignment");
constexpr int kNumBars = 2 * kMaxStages + 4 + 2 * kQueue + 1 + 2 * kBgStages + 2 + 2 * kBgQueue;
constexpr int kBarBytes = kBarBytesDecl;       // >= 8 * kNumBars, keeps the staging area 128-byte aligned
// Output staging of the epilogue: results go to shared memory and leave as bulk copies of one row each,
// so that the epilogue warps never wait on the global store path (which the operand loads saturate).
// Each group of four epilogue warps owns a quarter of it.
constexpr int kOutStageBytes = 32768;
constexpr int kEpiGroups = 4;                  // groups of four epilogue warps (one warp per TMEM lane quarter)
constexpr int kOutGroupBytes = kOutStageBytes / kEpiGroups;
constexpr int kSmemBytes = kRingBytes + 1024 /* alignment slack */ + kBarBytes + kOutStageBytes;
static_assert(8 * kNumBars <= kBarBytes, "barrier area too small");
static_assert(kBgRingsBytes <= kRingBytes + kOutStageBytes, "the two rings must fit the shared memory of the CTA");
constexpr int kEpiWarps = 4 * kEpiGroups;      // four warps per TMEM lane quarter, taking the 16-column chunks in turn
constexpr int kSchedWarp = 2 + kEpiWarps;      // warp 0: TMA (weights), warp 1: MMA + TMEM, warps 2..17: epilogue, warp 18: scheduler,
constexpr int kTokWarp = kSchedWarp + 1;       // warp 19: TMA (tokens)
constexpr int kThreads = 32 * (kTokWarp + 1);
// background pipeline (pair shape only): warp 20 = its TMA producer (and, in the leader CTA, its scheduler), warp 21 =
// its MMA lane, warps 22..25 = its epilogue (one warp per TMEM lane quarter)
constexpr int kBgProdWarp = kTokWarp + 1, kBgMmaWarp = kTokWarp + 2, kBgEpiWarp0 = kTokWarp + 3;
constexpr int kThreadsBg = 32 * (kBgEpiWarp0 + 4);
constexpr uint32_t kBgTmemCol = 2 * kBgAccRows;     // its accumulator: TMEM columns 448 .. 511
constexpr int kClaimAhead = 8;                 // the next unit is claimed this many K steps before the current one is loaded
constexpr uint32_t kTmemCols = 512;            // 2 accumulator buffers x 256 columns

struct GemmParams {
    const Unit* units;
    const int32_t* n_units;
    const int32_t* n_shared;      // shared-expert units at the head of the list that are to be spread evenly over the
                                  // launch (0: take the list in order)
    const int32_t* n_short;       // units at the tail of the list that the background lanes may take (0: none)
    unsigned long long* counter;  // work counter of the dynamic scheduler (zeroed by the plan kernel): units taken from
                                  // the front of the list in the low word, from its tail in the high word
    const Tile* tiles;
    const Tile* stiles;
    const int32_t* perm;          // direct mode: routed row -> flat (token, j) id
    int top_k;
    int direct;                   // 1: routed gate/up units read the tokens in place and pick their columns
    int n_tokens_pad;             // direct mode: tokens rounded up to 16
    int k_routed, k_shared;       // contraction lengths
    int rows_per_slot;            // weight rows per pool slot in the routed A map
    int cb_rows;                  // weight rows (gate/up: intermediate indices) per colblock: 64 or 128
    void* out_routed;
    void* out_shared;
    int ld_routed, ld_shared;
    const int32_t* shared_dst_rows;
    uint32_t idesc_fmt_routed, idesc_fmt_shared;   // operand format bits of the instruction descriptor
    uint32_t gate_first_routed;   // bit 0: the gate row is the even TMEM lane of a pair (routed map)
    uint32_t gate_first_shared;   // bit m: same for the shared expert of model m
    int stream_weights;           // 1: every weight tile is read once: mark it evict-first in L2
    int group;                    // stages handed back to the producer per commit (divides the stage count)
    int wide;                     // 1: tiles of up to 512 rows (pair shape only): 4 stages of 48 KB instead of 6 of 32 KB
    int head_units;               // token-major gate/up launch of a layer pass, one model, one token tile: the shared
                                  // expert's units at the head of the list (unit i = weight rows 256 i .. of all head_rows
                                  // tokens).  They depend on nothing the kernels before this one produce, so CTA b runs
                                  // units b, b + grid, ... of them before it waits for those kernels.  0: none.
    int head_rows;
    const void* pull_ptr;         // with head units: static bytes that the CTAs without a head unit pull into L2 before they
    unsigned long long pull_bytes;//   wait (the shared expert's down weights, which the next launch reads); 0: none
    int32_t* status;
};

constexpr int kTcMaxModels = 8;

// TMA descriptors in kernel-parameter space
struct GemmMaps {
    CUtensorMap a_routed[3];               // gate/up: 3-D (K, {gate,up}, S*I); down: 2-D (K, S*H); [1], [2]: boxes of a half
    CUtensorMap a_shared[kTcMaxModels][3]; //   and a quarter of the weight rows (token-major shape); same for the shared experts
    CUtensorMap b_routed[5];               // activations of the routed units, boxes of 128 / 64 / 32 / 16 rows, and of
    CUtensorMap b_shared[5];               //   kBgAccRows / 2 rows (one CTA's share of a full accumulator of the background shape)
};

__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "l"(policy)
        : "memory");
}
// pair mode: the load lands in this CTA's shared memory, its bytes are counted on the leader's barrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar & 0xFEFFFFFFu), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(map), "r"(bar & 0xFEFFFFFFu), "r"(x), "r"(y), "r"(z), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives on the barrier at the same offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3)
                 : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t& r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr));
}

// bulk copy shared -> global of one output row (16-byte aligned on both sides, size a multiple of 16)
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t ssrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// barrier of one epilogue group (128 threads) that also ANDs a flag over the group
__device__ __forceinline__ bool group_and(int id, bool v)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, %2, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)v), "r"(id) : "memory");
    return r != 0;
}
__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// The shared expert's SwiGLU activations are stored as fp16 (finer than bf16, but a range of only +-65504): a value
// beyond that range saturates instead of becoming infinite.  Activations of that size do not occur with weights and
// inputs of ordinary scale; every value inside the range is unchanged.
__device__ __forceinline__ float clamp_fp16(float v) { return fminf(fmaxf(v, -65504.f), 65504.f); }

struct UnitInfo {
    int a_row, amap;              // first weight row of the tile; -1: routed map, m: shared map of model m
    int b_row0, nrows, npad, ksteps, shared, cb, model;
    int npad1;                    // wide unit: padded rows of the second accumulator (rows 256..), else 0
    int width;                    // token-major shape: weight rows of the unit: 256, 128 or 64; a stage then holds 1, 2 or 4
    int kb;                       //   slices of 64 K elements (always 32 KB of weights), so that narrow units stream as fast
    int direct;                   // routed gate/up unit in direct mode: B = all tokens
};

// One slot of the unit queue: the unit as the scheduler decoded it for cluster rank 0, so that no other role
// has to chase the unit and tile tables through global memory.  u < 0: no more work.
struct __align__(16) QEntry {
    int u, tile_slot, b_row0, nrows;
    int colblock, shared, pad0, pad1;
};

template <int MODE, bool PAIR, bool SWAP, bool BG>
__device__ __forceinline__ UnitInfo unit_info(const GemmParams& p, const QEntry& e, uint32_t rank)
{
    UnitInfo ui;
    ui.shared = e.shared;
    ui.cb = PAIR ? 2 * e.colblock + (int)rank : e.colblock;      // (token-major shape: in steps of 64 weight rows)
    ui.width = SWAP ? e.pad0 : 0;
    ui.kb = SWAP ? 256 / e.pad0 : 1;
    ui.model = e.tile_slot;
    ui.amap = ui.shared ? e.tile_slot : -1;
    ui.a_row = (ui.shared ? 0 : e.tile_slot * p.rows_per_slot) + ui.cb * p.cb_rows;
    ui.b_row0 = e.b_row0;
    ui.nrows = e.nrows;
    ui.direct = (MODE == 0 && p.direct && !ui.shared) ? 1 : 0;
    ui.npad1 = 0;
    if (ui.direct) { ui.npad = p.n_tokens_pad; }
    else if (PAIR) {
        // wide tiles: the first kAcc rows go to one accumulator, the rest to the other
        constexpr int kAcc = BG ? kBgAccRows : 256;
        const int n0 = e.nrows < kAcc ? e.nrows : kAcc;
        ui.npad = (n0 + 31) & ~31;
        ui.npad1 = (e.nrows - n0 + 31) & ~31;
    }
    else ui.npad = (e.nrows + 15) & ~15;      // (token-major shape: rows of the token tile that are loaded)
    const int k_len = ui.shared ? p.k_shared : p.k_routed;
    // pair shape with 48 KB stages: a unit of at most 128 tokens puts two K slices into a stage (2 x 16 KB of weights
    // and 2 x at most 8 KB of tokens per CTA), which halves the waits and commits of its MMA lane -- all a short unit costs
    // (with the background pipeline the stages are 44 KB: two K slices fit up to 96 tokens)
    if (PAIR && p.wide && ui.npad1 == 0 && ui.npad <= (BG ? 96 : 128) && (k_len / kBK) % 2 == 0) ui.kb = 2;
    ui.ksteps = k_len / (kBK * ui.kb);
    return ui;
}

__device__ __forceinline__ QEntry read_entry(const QEntry* q)
{
    const int4 a = *reinterpret_cast<const int4*>(q);
    const int2 b = *reinterpret_cast<const int2*>(&q->colblock);
    QEntry e;
    e.u = a.x; e.tile_slot = a.y; e.b_row0 = a.z; e.nrows = a.w; e.colblock = b.x; e.shared = b.y; e.pad0 = q->pad0; e.pad1 = q->pad1;
    return e;
}

// The background pipeline of the pair shape: producer (+ scheduler in the leader CTA), MMA lane and epilogue warps for
// the short tiles (at most kShortRows tokens) at the tail of the unit list.  One K slice per stage (128 weight rows and
// at most 32 token rows per CTA), a ring of kBgStages stages, one accumulator of 64 TMEM columns.
template <int MODE>
__device__ __forceinline__ void bg_roles(const GemmParams& p, const GemmMaps& maps, int warp, int lane, uint32_t rank,
                                         uint32_t ring, uint32_t b_full, uint32_t b_empty, uint32_t b_tfull,
                                         uint32_t b_tempty, uint32_t b_qfull, uint32_t b_qempty, QEntry* queue,
                                         uint32_t tmem_base, int n_units, int n_short, int* s_abort)
{
    const bool leader = rank == 0;
    const uint32_t qempty_leader = map_to_cta(b_qempty, 0);
    const int ksteps = p.k_routed / kBK;
    if (warp == kBgProdWarp) {
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, q = 0, qphase = 0, armed = 0, armed_phase = 0;
            const uint64_t pol_w = l2_evict_first(), pol_x = l2_evict_last();
            const uint32_t peer_queue = map_to_cta(smem_u32(queue), 1), peer_qfull = map_to_cta(b_qfull, 1);
            bool ok = true;
            while (ok) {
                QEntry e;
                if (leader) {
                    // scheduler: a free queue slot, then a unit from the tail of the list (while short units are left
                    // there and the two ends have not met)
                    if (!mbar_wait_cluster(b_qempty + 8 * q, qphase ^ 1, s_abort, p.status)) { ok = false; break; }
                    int ix = -1;
                    for (;;) {
                        const unsigned long long w = *reinterpret_cast<volatile unsigned long long*>(p.counter);
                        const uint32_t f = (uint32_t)w, b = (uint32_t)(w >> 32);
                        if ((int)b >= n_short || (unsigned long long)f + b >= (unsigned long long)n_units) break;
                        if (atomicCAS(p.counter, w, w + (1ull << 32)) == w) { ix = n_units - 1 - (int)b; break; }
                    }
                    e.u = -1; e.tile_slot = 0; e.b_row0 = 0; e.nrows = 0; e.colblock = 0; e.shared = 0; e.pad0 = 0; e.pad1 = 0;
                    if (ix >= 0) {
                        const Unit un = p.units[ix];
                        const Tile t = p.tiles[un.tile];
                        e.u = ix; e.tile_slot = t.slot; e.b_row0 = t.row0; e.nrows = t.nrows; e.colblock = un.colblock & 0xffffff;
                    }
                    *reinterpret_cast<int4*>(&queue[q]) = make_int4(e.u, e.tile_slot, e.b_row0, e.nrows);
                    *reinterpret_cast<int2*>(&queue[q].colblock) = make_int2(e.colblock, 0);
                    queue[q].pad0 = 0;
                    mbar_arrive(b_qfull + 8 * q);
                    const uint32_t dst = peer_queue + (uint32_t)sizeof(QEntry) * q;
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(e.u), "r"(e.tile_slot),
                                 "r"(e.b_row0), "r"(e.nrows) : "memory");
                    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(dst + 16), "r"(e.colblock), "r"(0) : "memory");
                    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(dst + 24), "r"(0) : "memory");
                    mbar_arrive_cluster(peer_qfull + 8 * q);
                } else {
                    if (!mbar_wait_cluster(b_qfull + 8 * q, qphase, s_abort, p.status)) { ok = false; break; }
                    e = read_entry(&queue[q]);
                    mbar_arrive_cluster(qempty_leader + 8 * q);
                }
                if (++q == kBgQueue) { q = 0; qphase ^= 1; }
                if (e.u < 0) break;
                // this CTA's half of the unit: 128 weight rows, half of the (padded) token rows
                const int npad = (e.nrows + 31) & ~31;
                const int my_rows = npad >> 1;                                        // 16 or 32
                const int cb = 2 * e.colblock + (int)rank;
                const int a_row = e.tile_slot * p.rows_per_slot + cb * p.cb_rows;
                const int my_row0 = e.b_row0 + (int)rank * my_rows;
                const CUtensorMap* ma = &maps.a_routed[0];
                const CUtensorMap* mb = maps.b_routed + (my_rows == 32 ? 2 : 3);     // boxes of 32 / 16 rows
                for (int ks = 0; ks < ksteps; ++ks) {
                    if (!mbar_wait(b_empty + 8 * stage, phase ^ 1, s_abort, p.status)) { ok = false; break; }
                    const uint32_t sa = ring + stage * kBgStageBytes;
                    const uint32_t full = b_full + 8 * stage;
                    if (leader) mbar_expect_tx(full, 2u * (uint32_t)(kABytes + my_rows * kBK * 2));
                    armed |= 1u << stage;
                    armed_phase = (armed_phase & ~(1u << stage)) | (phase << stage);
                    if (MODE == 0) tma_load_3d_pair(sa, ma, full, ks * kBK, 0, a_row, pol_w);
                    else tma_load_2d_pair(sa, ma, full, ks * kBK, a_row, pol_w);
                    tma_load_2d_pair(sa + kABytes, mb, full, ks * kBK, my_row0, pol_x);
                    if (++stage == kBgStages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && leader) {
                // gave up: let the copies already in flight land before the block exits
                for (int s2 = 0; s2 < kBgStages; ++s2)
                    if (armed & (1u << s2)) mbar_wait(b_full + 8 * s2, (armed_phase >> s2) & 1u, s_abort, p.status);
            }
        }
        __syncwarp();
    } else if (warp == kBgMmaWarp) {
        if (lane == 0 && leader) {
            uint32_t stage = 0, phase = 0, q = 0, qphase = 0, tphase = 0;
            const uint32_t d = tmem_base + kBgTmemCol;
            bool ok = true;
            while (ok) {
                if (!mbar_wait(b_qfull + 8 * q, qphase, s_abort, p.status)) { ok = false; break; }
                const QEntry e = read_entry(&queue[q]);
                mbar_arrive(b_qempty + 8 * q);
                if (++q == kBgQueue) { q = 0; qphase ^= 1; }
                if (e.u < 0) break;
                const int npad = (e.nrows + 31) & ~31;
                const uint32_t idesc = (1u << 4) | p.idesc_fmt_routed | ((256u >> 4) << 24) | ((uint32_t)(npad >> 3) << 17);
                if (!mbar_wait_cluster(b_tempty, tphase ^ 1, s_abort, p.status)) { ok = false; break; }
                tc_fence_after();
                uint32_t acc = 0;
                for (int ks = 0; ks < ksteps; ++ks) {
                    if (!mbar_wait(b_full + 8 * stage, phase, s_abort, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t lo_m = smem_desc_lo(ring + stage * kBgStageBytes), lo_n = lo_m + (kABytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        umma_bf16_pair(d, smem_desc_pack(lo_m + 2 * kk), smem_desc_pack(lo_n + 2 * kk), idesc, acc);
                        acc = 1;
                    }
                    umma_commit_pair(b_empty + 8 * stage);
                    if (++stage == kBgStages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                umma_commit_pair(b_tfull);
                tphase ^= 1;
            }
        }
        __syncwarp();
    } else {
        // epilogue: one warp per TMEM lane quarter; results go straight to global memory (a few KB per unit)
        const int quarter = warp & 3;
        const uint32_t d = tmem_base + ((uint32_t)(quarter * 32) << 16) + kBgTmemCol;
        const uint32_t tempty_leader = map_to_cta(b_tempty, 0);
        uint32_t q = 0, qphase = 0, tphase = 0;
        bool ok = true;
        while (ok) {
            ok = __all_sync(0xffffffffu, mbar_wait_cluster(b_qfull + 8 * q, qphase, s_abort, p.status));
            if (!ok) break;
            const QEntry e = read_entry(&queue[q]);
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(qempty_leader + 8 * q);
            if (++q == kBgQueue) { q = 0; qphase ^= 1; }
            if (e.u < 0) break;
            ok = __all_sync(0xffffffffu, mbar_wait(b_tfull, tphase, s_abort, p.status));
            if (!ok) break;
            tphase ^= 1;
            tc_fence_after();
            const int cb = 2 * e.colblock + (int)rank;
            const int nchunk = ((e.nrows + 31) & ~31) >> 4;                 // 16-token chunks: 2 or 4
            if (MODE == 0) {
                // lanes 2i / 2i+1 hold the gate / up row (or up / gate) of intermediate index cb*64 + quarter*16 + i
                const bool even = (lane & 1) == 0;
                const bool own_is_gate = even == ((p.gate_first_routed & 1u) != 0);
                uint32_t o[16];                                             // 8 outputs of 16 bits per chunk
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (c < nchunk) {
                        uint32_t r[16];
                        tmem_ld16(d + c * 16, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            unsigned short h2[2];
#pragma unroll
                            for (int t = 0; t < 2; ++t) {
                                // the even lane finishes token c*16 + j + 2t, the odd lane the one after it
                                const float send = __uint_as_float(even ? r[j + 2 * t + 1] : r[j + 2 * t]);
                                const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                                const float own = __uint_as_float(even ? r[j + 2 * t] : r[j + 2 * t + 1]);
                                const float g = own_is_gate ? own : recv, up = own_is_gate ? recv : own;
                                h2[t] = __bfloat16_as_ushort(__float2bfloat16_rn(__fdividef(g, 1.f + __expf(-g)) * up));
                            }
                            o[c * 4 + (j >> 2)] = (uint32_t)h2[0] | ((uint32_t)h2[1] << 16);
                        }
                    }
                }
                // the accumulator is free as soon as it has been read
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(tempty_leader);
                unsigned short* out16 = reinterpret_cast<unsigned short*>(p.out_routed) + cb * 64 + quarter * 16 + (lane >> 1);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const int n = c * 16 + 2 * jj + (even ? 0 : 1);
                        if (c < nchunk && n < e.nrows)
                            out16[(size_t)(e.b_row0 + n) * p.ld_routed] = (unsigned short)(o[c * 4 + (jj >> 1)] >> ((jj & 1) * 16));
                    }
                }
            } else {
                // this thread's TMEM lane is output feature cb*128 + quarter*32 + lane; a chunk holds 16 tokens
                float* outp = reinterpret_cast<float*>(p.out_routed) + cb * 128 + quarter * 32 + lane;
                for (int c = 0; c < nchunk; ++c) {
                    uint32_t r[16];
                    tmem_ld16(d + c * 16, r);
                    tmem_ld_wait();
                    if (c == nchunk - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty_leader);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = c * 16 + j;
                        if (n < e.nrows) outp[(size_t)(e.b_row0 + n) * p.ld_routed] = __uint_as_float(r[j]);
                    }
                }
            }
        }
    }
}

// MODE 0: gate/up + SwiGLU (output bf16 for routed units, fp16 for shared units)
// MODE 1: down projection (output fp32)
// SWAP (one CTA per unit only): the tokens are the M operand (one TMEM lane per token, up to 128) and up to 256
// weight rows the N operand.  One MMA then covers twice the weight bytes of the other orientation, which is what
// counts for short tiles: an MMA costs its issuing lane about 100 cycles however narrow it is, so with weights as M
// a tile of a few tokens is bound by MMA issue, not by the weight stream.
// BG (pair shape only): a second, small pipeline beside the main one.  A short tile (at most kShortRows tokens) costs the
// main MMA lane about as many issue slots as a tile of hundreds of tokens, while it hardly loads the tensor pipe; and
// while a CTA pair works through it, its share of the HBM stream is all it uses.  So the short tiles sit at the tail of
// the unit list, and every CTA pair has a background TMA lane, MMA lane, 60 KB stage ring and 64-column accumulator
// that take units from that tail while the main lanes take units from the front: the short tiles' weights stream in
// behind the tensor-bound tiles.  Whichever side reaches the other's end of the list first stops there (one packed
// counter orders all claims), so the main lanes finish whatever short tiles are left.  Every output element is still
// accumulated over K in the same order by one lane: results do not depend on which pipeline ran a unit.
template <int MODE, bool PAIR, bool SWAP, bool BG>
__global__ void __launch_bounds__(BG ? kThreadsBg : kThreads, 1)
grouped_gemm_kernel(const GemmParams p, const __grid_constant__ GemmMaps maps)
{
    static_assert(!(PAIR && SWAP), "the token-major shape is a one-CTA shape");
    static_assert(PAIR || !BG, "the background pipeline belongs to the pair shape");
    constexpr int kAcc = BG ? kBgAccRows : 256;                               // token rows (TMEM columns) per accumulator
    constexpr uint32_t kAccBytes = (uint32_t)(kAcc / 2) * kBK * 2;            // pair shape: token tile of one CTA per accumulator
    constexpr uint32_t kWBytes = SWAP ? 2 * kABytes : kABytes;               // weight tile of one stage
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
    const uint32_t bars = smem_base + (BG ? kBgRingsBytes : kRingBytes);       // 8-byte barriers after the tiles
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kMaxStages;
    const uint32_t bar_tfull = bars + 16 * kMaxStages, bar_tempty = bar_tfull + 16;
    const uint32_t n_stages = BG ? kBgMainStages : (((PAIR && p.wide) || SWAP) ? kWideStages : kMaxStages);
    const uint32_t stage_bytes = BG ? kBgStageBytesMain : kRingBytes / n_stages;
    // Stages are handed back to the producer in groups: a tcgen05.commit costs the issuing lane about as much
    // as two MMAs, so with four MMAs per stage one commit per stage would starve the tensor pipe.
    const uint32_t group = (uint32_t)p.group;                                  // 1 or 2: masks and shifts below, a
    const uint32_t gmask = group - 1, gshift = group >> 1;                     // division per K step would be felt
    const uint32_t bar_qfull = bar_tempty + 16, bar_qempty = bar_qfull + 8 * kQueue;
    const uint32_t bar_sched = bar_qempty + 8 * kQueue;
    // background pipeline: stage barriers, accumulator barriers, unit queue; its ring follows the main one
    const uint32_t bg_full = bar_sched + 8, bg_empty = bg_full + 8 * kBgStages;
    const uint32_t bg_tfull = bg_empty + 8 * kBgStages, bg_tempty = bg_tfull + 8;
    const uint32_t bg_qfull = bg_tempty + 8, bg_qempty = bg_qfull + 8 * kBgQueue;
    const uint32_t bg_ring = smem_base + kBgMainStages * kBgStageBytesMain;
    __shared__ QEntry s_bg_queue[kBgQueue];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ QEntry s_queue[kQueue];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, (PAIR ? 2 : 1) * kEpiWarps); }
        // unit queue: filled by the scheduler lane (of the leader CTA); drained by the two producer lanes, the MMA lane
        // and the epilogue warps of this CTA and, in pair mode, by the peer's producer lanes and epilogue warps
        for (int q = 0; q < kQueue; ++q) {
            mbar_init(bar_qfull + 8 * q, 1);
            mbar_init(bar_qempty + 8 * q, 3 + kEpiWarps + (PAIR ? 2 + kEpiWarps : 0));
        }
        mbar_init(bar_sched, 1);
        if (BG) {
            for (int s2 = 0; s2 < kBgStages; ++s2) { mbar_init(bg_full + 8 * s2, 1); mbar_init(bg_empty + 8 * s2, 1); }
            mbar_init(bg_tfull, 1);
            mbar_init(bg_tempty, 2 * 4);                  // the four background epilogue warps of both CTAs
            // unit queue: filled by the leader's background producer (which is the scheduler); drained by the leader's
            // MMA lane and epilogue warps and by the peer's producer and epilogue warps
            for (int q2 = 0; q2 < kBgQueue; ++q2) { mbar_init(bg_qfull + 8 * q2, 1); mbar_init(bg_qempty + 8 * q2, 1 + 4 + 1 + 4); }
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                         "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                         "r"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();          // the peer's barriers are initialised before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    // Set-up above overlaps the previous kernel; its results are read from here on.  The down projection follows the
    // gate/up launch, which had itself waited for the plan before it let this kernel start: the unit lists are
    // complete, and the scheduler and the weight producer (static data) go ahead and fill the ring while the token
    // producer and the epilogue wait for the activations.
    // A gate/up launch with head units (see GemmParams) starts on them at once -- while the router and the dispatch
    // are still running -- and every role waits when it meets the first unit of the work plan.  Such a launch lets the
    // down projection start only after the scheduler has waited: that kernel relies on the plan being complete.
    const bool head = MODE == 0 && SWAP && !PAIR && p.head_units > 0;
    if (!head) {
        if (!(MODE == 1 && (warp == 0 || warp == kSchedWarp))) pdl_wait();
        pdl_launch_dependents();
    }
    const int n_units = head ? 0 : *p.n_units;            // (with head units the scheduler reads the counts after its wait)
    const int n_shared = head ? 0 : *p.n_shared;
    const int n_short = (BG && !head) ? *p.n_short : 0;

    // Units are pulled from a global counter by one scheduler lane per CTA (pair: per CTA pair, the leader's),
    // decoded, and handed to the other roles through a small queue in shared memory; in pair mode the scheduler
    // also writes the peer's queue and the peer's consumers release the slot on the leader's barrier.  The
    // scheduler is a warp of its own: a global load or atomic issued by the lane that feeds the TMA unit
    // queues behind the tile requests and was measured to cost thousands of cycles per unit.
    const uint32_t qempty_leader = PAIR ? map_to_cta(bar_qempty, 0) : bar_qempty;

    if (warp == 0 || warp == kTokWarp) {
        // ---------------- TMA producers: one lane of warp 0 posts the byte count of a stage and loads the weight tile,
        // one lane of another warp loads the token tiles.  A tile load costs its issuing lane about 140 cycles and
        // the barrier handshake of a stage about 290, whatever the tile's size; in one lane that was more per K step
        // than the MMAs of a full tile take.  Lanes of one warp would not help: their branches run one after the other.
        const bool wrole = warp == 0;
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, q = 0, qphase = 0;
            uint32_t armed = 0, armed_phase = 0;
            bool ok = true, planned = false;
            const uint64_t pol_first = l2_evict_first(), pol_last = l2_evict_last();
            const uint64_t pol_x = l2_evict_last();
            while (ok) {
                if (!(leader ? mbar_wait(bar_qfull + 8 * q, qphase, &s_abort, p.status)
                             : mbar_wait_cluster(bar_qfull + 8 * q, qphase, &s_abort, p.status))) { ok = false; break; }
                const QEntry e = read_entry(&s_queue[q]);
                if (leader) mbar_arrive(bar_qempty + 8 * q); else mbar_arrive_cluster(qempty_leader + 8 * q);
                if (++q == kQueue) { q = 0; qphase ^= 1; }
                if (head && !planned && e.pad1) { pdl_wait(); planned = true; }     // the first unit (or the end mark) of the plan
                if (e.u < 0) break;
                const UnitInfo ui = unit_info<MODE, PAIR, SWAP, BG>(p, e, rank);
                const int claim_ks = ui.ksteps > kClaimAhead ? ui.ksteps - kClaimAhead : 0;
                // L2 policy of the weight tiles: a routed expert with at most 128 rows is read by one tile only, so its
                // weights stream through (evict-first) and leave the cache to what is read again -- the shared expert's
                // weights (every token tile of the model reads them) and the weights of the experts with several tiles
                const uint64_t pol_w = (p.stream_weights || (!ui.shared && ui.nrows <= 128)) ? pol_first : pol_last;
                const int wsel = SWAP ? (ui.width == 256 ? 0 : (ui.width == 128 ? 1 : 2)) : 0;
                const CUtensorMap* ma = ui.amap < 0 ? &maps.a_routed[wsel] : &maps.a_shared[ui.amap][wsel];
                const bool bshared = ui.shared || ui.direct;
                const CUtensorMap* mb = bshared ? maps.b_shared : maps.b_routed;
                const int brow0 = ui.direct ? 0 : ui.b_row0;
                const int my_rows = PAIR ? (ui.npad >> 1) : ui.npad;          // token rows this CTA loads
                const int my_row0 = brow0 + (PAIR ? (int)rank * my_rows : 0);
                const int my_rows1 = ui.npad1 >> 1;                           // same for the second accumulator
                const int my_row1 = brow0 + kAcc + (int)rank * my_rows1;
                for (int ks = 0; ks < ui.ksteps; ++ks) {
                    if (wrole && leader && ks == claim_ks) mbar_arrive(bar_sched);      // time to claim the next unit
                    if ((stage & gmask) == 0 &&
                        !mbar_wait(bar_empty + 8 * (stage >> gshift), phase ^ 1, &s_abort, p.status)) { ok = false; break; }
                    const uint32_t sa = smem_base + stage * stage_bytes, sb = sa + kWBytes;
                    const uint32_t full = bar_full + 8 * stage;
                    if (wrole) {
                        // the token lane's bytes may be counted before this is posted: the phase still cannot complete
                        // without this arrival
                        if (leader) mbar_expect_tx(full, (PAIR ? 2u : 1u) * (uint32_t)((PAIR ? ui.kb * kABytes : kWBytes) +
                                                                                       ui.kb * (my_rows + my_rows1) * kBK * 2));
                        armed |= 1u << stage;
                        armed_phase = (armed_phase & ~(1u << stage)) | (phase << stage);
                        if (PAIR) {
                            for (int a = 0; a < ui.kb; ++a) {
                                if (MODE == 0) tma_load_3d_pair(sa + a * kABytes, ma, full, (ks * ui.kb + a) * kBK, 0, ui.a_row, pol_w);
                                else tma_load_2d_pair(sa + a * kABytes, ma, full, (ks * ui.kb + a) * kBK, ui.a_row, pol_w);
                            }
                        } else {
                            // (token-major: kb slices of 64 K elements, each `width` rows high, one after the other)
                            for (int a = 0; a < ui.kb; ++a) {
                                const uint32_t dst = sa + (uint32_t)(a * ui.width) * kBK * 2;
                                if (MODE == 0) tma_load_3d_hint(dst, ma, full, (ks * ui.kb + a) * kBK, 0, ui.a_row, pol_w);
                                else tma_load_2d_hint(dst, ma, full, (ks * ui.kb + a) * kBK, ui.a_row, pol_w);
                            }
                        }
                    } else {
                        // token rows in boxes of 128 / 64 / 32 / 16 rows
                        const bool by_acc = PAIR && ui.kb == 1;
                        for (int acc = 0; acc < (by_acc ? 2 : ui.kb); ++acc) {
                            // pair shape: the two accumulators' tiles, or the K slices of a short unit (behind its two weight
                            // slices); token-major shape: the K slices of the stage
                            const int rows = (by_acc && acc) ? my_rows1 : my_rows, r0 = (by_acc && acc) ? my_row1 : my_row0;
                            const uint32_t dst = by_acc ? sb + acc * kAccBytes
                                                        : (PAIR ? sa + ui.kb * kABytes : sb) + acc * my_rows * kBK * 2;
                            const int kx = (by_acc ? ks : ks * ui.kb + acc) * kBK;
                            int j = 0;
                            if (BG && rows == kBgAccRows / 2) {
                                // a full accumulator of the background shape: one box (a load costs its issuing lane about
                                // 140 cycles; three boxes per accumulator and stage would make this lane the bottleneck)
                                tma_load_2d_pair(dst, mb + 4, full, kx, r0, pol_x);
                                j = rows;
                            }
#pragma unroll
                            for (int bx = 0; bx < 4; ++bx) {
                                const int n = 128 >> bx;
                                while (j + n <= rows) {
                                    if (PAIR) tma_load_2d_pair(dst + j * kBK * 2, mb + bx, full, kx, r0 + j, pol_x);
                                    else tma_load_2d_hint(dst + j * kBK * 2, mb + bx, full, kx, r0 + j, pol_x);
                                    j += n;
                                }
                            }
                        }
                    }
                    if (++stage == n_stages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && leader && wrole) {
                // gave up: let the copies already in flight land before the block exits
                for (int s = 0; s < kMaxStages; ++s)
                    if (armed & (1u << s)) mbar_wait(bar_full + 8 * s, (armed_phase >> s) & 1u, &s_abort, p.status);
            }
        }
        __syncwarp();      // the whole warp reaches the block barrier below together
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane; in pair mode only the leader CTA issues) ----------------
        if (lane == 0 && leader) {
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0, q = 0, qphase = 0;
            bool ok = true;
            while (ok) {
                if (!mbar_wait(bar_qfull + 8 * q, qphase, &s_abort, p.status)) { ok = false; break; }
                const QEntry e = read_entry(&s_queue[q]);
                mbar_arrive(bar_qempty + 8 * q);
                if (++q == kQueue) { q = 0; qphase ^= 1; }
                if (e.u < 0) break;
                const UnitInfo ui = unit_info<MODE, PAIR, SWAP, BG>(p, e, rank);
                const uint32_t fmt = ui.shared ? p.idesc_fmt_shared : p.idesc_fmt_routed;
                const uint32_t idesc_m = (1u << 4) | fmt | (((PAIR ? 256u : 128u) >> 4) << 24);
                const uint32_t idesc = idesc_m | ((uint32_t)((SWAP ? ui.width : ui.npad) >> 3) << 17);
                const uint32_t idesc1 = idesc_m | ((uint32_t)(ui.npad1 >> 3) << 17);
                const bool wide = PAIR && ui.npad1 > 0;
                // a wide unit takes both accumulator buffers, in the order the epilogue drains them
                if (!(PAIR ? mbar_wait_cluster(bar_tempty + 8 * buf, bphase ^ 1, &s_abort, p.status)
                           : mbar_wait(bar_tempty + 8 * buf, bphase ^ 1, &s_abort, p.status))) { ok = false; break; }
                const uint32_t d = tmem_base + buf * kAcc;
                const uint32_t buf1 = buf ^ 1u, bphase1 = buf ? (bphase ^ 1u) : bphase;
                const uint32_t d1 = tmem_base + buf1 * kAcc;
                tc_fence_after();
                // This lane is alone in its warp: every instruction of the loop below is paid in full, so whatever
                // does not change inside a unit is worked out here, and the descriptors are put together from two
                // 32-bit words (only the start-address field in the low word changes).
                //   slice step of the M operand / of the N operand inside a stage, in 16-byte units:
                const uint32_t m_step = (PAIR ? kABytes : (SWAP ? ui.npad * kBK * 2 : 0)) >> 4;
                const uint32_t n_step = (PAIR ? (ui.npad >> 1) * kBK * 2 : (SWAP ? ui.width * kBK * 2 : 0)) >> 4;
                //   pair shape, short unit: the token slices sit behind the two weight slices
                const uint32_t n_base = PAIR ? ((ui.kb - 1) * kABytes) >> 4 : 0;
                const uint32_t m_off = (SWAP ? kWBytes : 0) >> 4, n_off = (SWAP ? 0 : kWBytes) >> 4;
                uint32_t acc = 0;                                 // the first MMA of a unit overwrites the accumulator
                uint32_t acc1 = 0;
                for (int ks = 0; ks < ui.ksteps; ++ks) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, &s_abort, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t lo = smem_desc_lo(smem_base + stage * stage_bytes);
                    uint32_t lo_m = lo + m_off, lo_n = lo + n_off + n_base;
                    for (int a = 0; a < ui.kb; ++a) {
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk) {
                            // 16 elements = 32 bytes along K = 2 address units
                            if (PAIR) umma_bf16_pair(d, smem_desc_pack(lo_m + 2 * kk), smem_desc_pack(lo_n + 2 * kk), idesc, acc);
                            else umma_bf16(d, smem_desc_pack(lo_m + 2 * kk), smem_desc_pack(lo_n + 2 * kk), idesc, acc);
                            acc = 1;
                        }
                        lo_m += m_step; lo_n += n_step;
                    }
                    if (wide) {
                        if (ks == ui.ksteps - 1) umma_commit_pair(bar_tfull + 8 * buf);      // first half done: its epilogue may start
                        if (ks == 0) {
                            if (!mbar_wait_cluster(bar_tempty + 8 * buf1, bphase1 ^ 1, &s_abort, p.status)) { ok = false; break; }
                            tc_fence_after();
                        }
                        const uint32_t lo_m1 = lo + m_off, lo_n1 = lo + n_off + (kAccBytes >> 4);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk) {
                            umma_bf16_pair(d1, smem_desc_pack(lo_m1 + 2 * kk), smem_desc_pack(lo_n1 + 2 * kk), idesc1, acc1);
                            acc1 = 1;
                        }
                    }
                    // frees the stage group (in both CTAs of a pair) when these MMAs have read it
                    if ((stage & gmask) == gmask) {
                        if (PAIR) umma_commit_pair(bar_empty + 8 * (stage >> gshift)); else umma_commit(bar_empty + 8 * (stage >> gshift));
                    }
                    if (++stage == n_stages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                if (wide) {
                    umma_commit_pair(bar_tfull + 8 * buf1);
                    bphase ^= 1;                                   // two buffers taken: same buffer next, other phase
                } else {
                    if (PAIR) umma_commit_pair(bar_tfull + 8 * buf); else umma_commit(bar_tfull + 8 * buf);
                    if (++buf == 2) { buf = 0; bphase ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp < kSchedWarp) {
        // ---------------- epilogue: two groups of four warps (one warp per TMEM lane quarter), ----------------
        // ---------------- the groups alternate over the 16-column chunks of an accumulator     ----------------
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;                  // group: 0 .. kEpiGroups - 1
        const int gbar = 1 + half;                         // named barrier of the group
        const int gtid = quarter * 32 + lane;              // thread index inside the group
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const uint32_t stg = bars + kBarBytes + half * kOutGroupBytes;      // this group's staging area
        uint32_t buf = 0, bphase = 0, q = 0, qphase = 0;
        bool ok = true, planned = false;
        const uint32_t tempty_leader = PAIR ? map_to_cta(bar_tempty, 0) : bar_tempty;
        while (ok) {
            ok = __all_sync(0xffffffffu, PAIR ? mbar_wait_cluster(bar_qfull + 8 * q, qphase, &s_abort, p.status)
                                              : mbar_wait(bar_qfull + 8 * q, qphase, &s_abort, p.status));
            if (!ok) break;
            const QEntry e = read_entry(&s_queue[q]);
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(qempty_leader + 8 * q); else mbar_arrive(bar_qempty + 8 * q);
            }
            if (++q == kQueue) { q = 0; qphase ^= 1; }
            if (head && !planned && e.pad1) { pdl_wait(); planned = true; }         // (warp-uniform)
            if (e.u < 0) break;
            const UnitInfo ui = unit_info<MODE, PAIR, SWAP, BG>(p, e, rank);
            const int ld = ui.shared ? p.ld_shared : p.ld_routed;
            const int n_acc = (PAIR && ui.npad1 > 0) ? 2 : 1;
            for (int hh = 0; hh < n_acc && ok; ++hh) {
                // rows of this accumulator: a wide unit keeps rows 256.. in its second one
                const int row0 = ui.b_row0 + hh * kAcc;
                const int nrows = hh ? ui.nrows - kAcc : (n_acc == 2 ? kAcc : ui.nrows);
                const int npad = hh ? ui.npad1 : ui.npad;
                ok = mbar_wait(bar_tfull + 8 * buf, bphase, &s_abort, p.status);
                const uint32_t d = tmem_base + lane_addr + buf * kAcc;
                if (SWAP) {
                    // Token-major accumulator: this thread's TMEM lane is token `gtid` of the tile, the columns are the
                    // unit's weight rows (256, 128 or 64); each group takes a quarter of them.  Every thread stages and
                    // sends only its own token's outputs (a 64-byte slot), so the group needs no barrier.
                    const int gcols = ui.width / kEpiGroups;  // columns of this group: 64, 32 or 16
                    const int c_first = half * gcols;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    // destination row of this thread's token, -1: none
                    int drow = -1;
                    if (ui.direct) {
                        // the tile holds all tokens; this expert's rows name theirs through perm
                        for (int j = 0; j < nrows; ++j)
                            if (p.perm[row0 + j] / p.top_k == gtid) drow = row0 + j;
                    } else if (gtid < nrows) {
                        drow = row0 + gtid;
                    }
                    if (MODE == 0) {
                        // columns 2i / 2i+1 hold the gate / up row (or up / gate) of intermediate index cb*32 + i
                        const uint32_t gf = ui.shared ? (p.gate_first_shared >> ui.model) & 1u : p.gate_first_routed & 1u;
                        const uint32_t mine = stg + (uint32_t)gtid * 64u;        // up to 32 outputs of 16 bits
                        bulk_wait_read<0>();                                     // the row sent for the previous tile has left
#pragma unroll 2
                        for (int i = 0; i < (gcols >> 4); ++i) {
                            uint32_t r[16];
                            tmem_ld16(d + c_first + i * 16, r);
                            tmem_ld_wait();
                            uint32_t o[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                unsigned short h2[2];
#pragma unroll
                                for (int t = 0; t < 2; ++t) {
                                    const float a = __uint_as_float(r[4 * j + 2 * t]), b = __uint_as_float(r[4 * j + 2 * t + 1]);
                                    const float g = gf ? a : b, up = gf ? b : a;
                                    const float v = __fdividef(g, 1.f + __expf(-g)) * up;
                                    h2[t] = ui.shared ? __half_as_ushort(__float2half_rn(clamp_fp16(v))) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
                                }
                                o[j] = (uint32_t)h2[0] | ((uint32_t)h2[1] << 16);
                            }
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(mine + i * 16), "r"(o[0]), "r"(o[1]), "r"(o[2]),
                                         "r"(o[3]) : "memory");
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                        fence_async_smem();
                        if (drow >= 0) {
                            unsigned short* out16 = reinterpret_cast<unsigned short*>(ui.shared ? p.out_shared : p.out_routed);
                            bulk_store(out16 + (size_t)drow * ld + ui.cb * 32 + (c_first >> 1), mine, (uint32_t)gcols);
                        }
                        bulk_commit();
                    } else {
                        // fp32 outputs, 16 at a time through this thread's 64-byte slot
                        if (drow >= 0 && ui.shared && p.shared_dst_rows != nullptr) drow = p.shared_dst_rows[drow];
                        float* outp = reinterpret_cast<float*>(ui.shared ? p.out_shared : p.out_routed) + ui.cb * 64 + c_first;
                        const int nchunk = gcols >> 4;
                        const uint32_t slot = stg + (uint32_t)gtid * 64u;
                        for (int i = 0; i < nchunk; ++i) {
                            bulk_wait_read<0>();
                            uint32_t r[16];
                            tmem_ld16(d + c_first + i * 16, r);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slot + j * 16), "r"(r[4 * j]), "r"(r[4 * j + 1]),
                                             "r"(r[4 * j + 2]), "r"(r[4 * j + 3]) : "memory");
                            if (i == nchunk - 1) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                            }
                            fence_async_smem();
                            if (drow >= 0) bulk_store(outp + (size_t)drow * ld + i * 16, slot, 64u);
                            bulk_commit();
                        }
                    }
                } else if (MODE == 0 && ui.direct) {
                    // one decision for the whole warp: the TMEM loads below are warp-wide instructions
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    // lanes 2i / 2i+1 hold the gate / up row (or up / gate) of intermediate index cb*64 + quarter*16 + i
                    const bool even = (lane & 1) == 0;
                    const bool own_is_gate = even == ((p.gate_first_routed & 1u) != 0);
                    const int col = ui.cb * 64 + quarter * 16 + (lane >> 1);
                    for (int j = half; j < nrows; j += kEpiGroups) {
                        const int tok = p.perm[row0 + j] / p.top_k;            // warp-uniform
                        uint32_t r;
                        tmem_ld1(d + tok, r);
                        tmem_ld_wait();
                        const float own = __uint_as_float(r);
                        const float other = __shfl_xor_sync(0xffffffffu, own, 1);
                        if (even) {
                            const float g = own_is_gate ? own : other, up = own_is_gate ? other : own;
                            reinterpret_cast<bf16*>(p.out_routed)[(size_t)(row0 + j) * ld + col] =
                                __float2bfloat16_rn(__fdividef(g, 1.f + __expf(-g)) * up);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                } else if (BG && MODE == 0) {
                    // (background shape: no staging area) every thread writes its own results; the accumulator is
                    // released as soon as its last chunk is in registers
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t gf = ui.shared ? (p.gate_first_shared >> ui.model) & 1u : p.gate_first_routed & 1u;
                    const bool even = (lane & 1) == 0;
                    const bool own_is_gate = even == (gf != 0);
                    // lanes 2i / 2i+1 hold the gate / up row (or up / gate) of intermediate index cb*64 + quarter*16 + i
                    unsigned short* out16 = reinterpret_cast<unsigned short*>(ui.shared ? p.out_shared : p.out_routed) +
                                            ui.cb * 64 + quarter * 16 + (lane >> 1);
                    bool released = false;
                    for (int c0 = half * 16; c0 < npad; c0 += 16 * kEpiGroups) {
                        uint32_t r[16];
                        tmem_ld16(d + c0, r);
                        tmem_ld_wait();
                        if (c0 + 16 * kEpiGroups >= npad) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
                            released = true;
                        }
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            // the even lane finishes token c0+j, the odd lane token c0+j+1
                            const float send = __uint_as_float(even ? r[j + 1] : r[j]);
                            const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                            const float own = __uint_as_float(even ? r[j] : r[j + 1]);
                            const float g = own_is_gate ? own : recv, up = own_is_gate ? recv : own;
                            const float v = __fdividef(g, 1.f + __expf(-g)) * up;
                            const unsigned short o = ui.shared ? __half_as_ushort(__float2half_rn(clamp_fp16(v)))
                                                               : __bfloat16_as_ushort(__float2bfloat16_rn(v));
                            const int n = c0 + j + (even ? 0 : 1);
                            if (n < nrows) out16[(size_t)(row0 + n) * ld] = o;
                        }
                    }
                    if (!released) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
                    }
                } else if (BG) {
                    // fp32 results: this thread's TMEM lane is output feature cb*128 + quarter*32 + lane, so the lanes
                    // of a warp write 128 contiguous bytes per token
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const bool remap = ui.shared && p.shared_dst_rows != nullptr;
                    float* outp = reinterpret_cast<float*>(ui.shared ? p.out_shared : p.out_routed) + ui.cb * 128 + quarter * 32 + lane;
                    bool released = false;
                    for (int c0 = half * 16; c0 < npad; c0 += 16 * kEpiGroups) {
                        uint32_t r[16];
                        tmem_ld16(d + c0, r);
                        tmem_ld_wait();
                        if (c0 + 16 * kEpiGroups >= npad) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
                            released = true;
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int n = c0 + j;
                            if (n < nrows) {
                                int row = row0 + n;
                                if (remap) row = p.shared_dst_rows[row];
                                outp[(size_t)row * ld] = __uint_as_float(r[j]);
                            }
                        }
                    }
                    if (!released) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
                    }
                } else if (MODE == 0) {
                    // The group's staging area holds its 4 chunks of 16 tokens as rows of 64 outputs (128 bytes).
                    // Its previous contents must have left (every thread waits for the rows it sent itself), and the
                    // whole group takes one decision on the accumulator wait.
                    bulk_wait_read<0>();
                    ok = group_and(gbar, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t gf = ui.shared ? (p.gate_first_shared >> ui.model) & 1u : p.gate_first_routed & 1u;
                    const bool even = (lane & 1) == 0;
                    const bool own_is_gate = even == (gf != 0);
                    // lanes 2i / 2i+1 hold the gate / up row (or up / gate) of intermediate index cb*64 + quarter*16 + i
                    const uint32_t my_col = stg + (uint32_t)(quarter * 32 + (lane >> 1) * 2);
                    int i = 0;
                    for (int c0 = half * 16; c0 < npad; c0 += 16 * kEpiGroups, ++i) {
                        uint32_t r[16];
                        tmem_ld16(d + c0, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            // the even lane finishes token c0+j, the odd lane token c0+j+1
                            const float send = __uint_as_float(even ? r[j + 1] : r[j]);
                            const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                            const float own = __uint_as_float(even ? r[j] : r[j + 1]);
                            const float g = own_is_gate ? own : recv, up = own_is_gate ? recv : own;
                            const float v = __fdividef(g, 1.f + __expf(-g)) * up;
                            const unsigned short o = ui.shared ? __half_as_ushort(__float2half_rn(clamp_fp16(v)))
                                                               : __bfloat16_as_ushort(__float2bfloat16_rn(v));
                            const uint32_t a = my_col + (uint32_t)(i * 16 + j + (even ? 0 : 1)) * 128u;
                            asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"(o) : "memory");
                        }
                    }
                    // the accumulator is free as soon as it has been read
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR) mbar_arrive_cluster(tempty_leader + 8 * buf); else mbar_arrive(bar_tempty + 8 * buf);
                    }
                    fence_async_smem();
                    group_sync(gbar);
                    // thread t < 64 of the group sends staged row t: token (t / 16) * 64 + group * 16 + t % 16
                    {
                        const int n = (gtid >> 4) * (16 * kEpiGroups) + half * 16 + (gtid & 15);
                        if (gtid < 64 && n < nrows) {
                            unsigned short* out16 = reinterpret_cast<unsigned short*>(ui.shared ? p.out_shared : p.out_routed);
                            bulk_store(out16 + (size_t)(row0 + n) * ld + ui.cb * 64, stg + (uint32_t)gtid * 128u, 128u);
                        }
                        bulk_commit();
                    }
                } else {
                    // fp32 rows of 128 outputs (512 bytes); a chunk of 16 tokens fills the group's staging area
                    const bool remap = ui.shared && p.shared_dst_rows != nullptr;
                    float* outp = reinterpret_cast<float*>(ui.shared ? p.out_shared : p.out_routed) + ui.cb * 128;
                    bool first = true;
                    const uint32_t slot = stg;
                    for (int c0 = half * 16; c0 < npad; c0 += 16 * kEpiGroups) {
                        bulk_wait_read<0>();                       // the rows this thread sent from the area have left
                        if (first) {
                            ok = group_and(gbar, ok);
                            if (!ok) break;
                            tc_fence_after();
                            first = false;
                        } else {
                            group_sync(gbar);
                        }
                        uint32_t r[16];
                        tmem_ld16(d + c0, r);
                        tmem_ld_wait();
                        const uint32_t a = slot + (uint32_t)(quarter * 128 + lane * 4);
#pragma unroll
                        for (int j = 0; j < 16; ++j) asm volatile("st.shared.b32 [%0], %1;" ::"r"(a + j * 512u), "r"(r[j]) : "memory");
                        if (c0 + 16 * kEpiGroups >= npad) {
                            // last chunk of this group: the accumulator has been read
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) {
                                if (PAIR) mbar_arrive_cluster(tempty_leader + 8 * buf); else mbar_arrive(bar_tempty + 8 * buf);
                            }
                        }
                        fence_async_smem();
                        group_sync(gbar);
                        if (lane < 4) {
                            const int j = quarter * 4 + lane, n = c0 + j;
                            if (n < nrows) {
                                int row = row0 + n;
                                if (remap) row = p.shared_dst_rows[row];
                                bulk_store(outp + (size_t)row * ld, slot + (uint32_t)j * 512u, 512u);
                            }
                        }
                        bulk_commit();
                    }
                    if (!ok) break;
                    if (first) {
                        // no chunk for this group (a tile with few columns): only release the accumulator
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        if (lane == 0) {
                            if (PAIR) mbar_arrive_cluster(tempty_leader + 8 * buf); else mbar_arrive(bar_tempty + 8 * buf);
                        }
                    }
                }
                if (++buf == 2) { buf = 0; bphase ^= 1; }
            }
        }
        bulk_wait_read<0>();       // staged rows are read before the block's shared memory goes away
    } else if (warp == kSchedWarp) {
        // ---------------- scheduler (one lane of the leader CTA) ----------------
        if (lane == 0 && leader) {
            uint32_t q = 0, qphase = 0, sphase = 0;
            bool first = true, planned = !head;
            int head_next = head ? (int)blockIdx.x : 0;
            int nu = n_units, nsh = n_shared;         // unit counts of the plan (read after the wait when there are head units)
            const uint32_t peer_queue = PAIR ? map_to_cta(smem_u32(&s_queue[0]), 1) : 0u;
            const uint32_t peer_qfull = PAIR ? map_to_cta(bar_qfull, 1) : 0u;
            for (;;) {
                // the first unit at once, every further one when the producer nears the end of its current unit
                if (!first) {
                    if (!mbar_wait(bar_sched, sphase, &s_abort, p.status)) break;
                    sphase ^= 1;
                }
                first = false;
                if (!(PAIR ? mbar_wait_cluster(bar_qempty + 8 * q, qphase ^ 1, &s_abort, p.status)
                           : mbar_wait(bar_qempty + 8 * q, qphase ^ 1, &s_abort, p.status))) break;
                // one packed counter orders the claims of both ends of the list: a claim is good while fewer than n_units
                // units have been taken in all
                int4 e0 = make_int4(-1, 0, 0, 0);
                int2 e1 = make_int2(0, 0);
                int e0w = 0;                  // token-major shape: weight rows of the unit
                int from_plan = 1;
                int u = 0;
                bool good = false;
                if (head && head_next < p.head_units) {
                    // a head unit: the shared expert's weight rows 256 i .. against all tokens (what the plan's list holds
                    // at index i, written out here because the plan may not exist yet)
                    u = head_next;
                    head_next += (int)gridDim.x;
                    e0 = make_int4(u, 0, 0, p.head_rows);
                    e1 = make_int2(u * 4, 1);
                    e0w = 256;
                    from_plan = 0;
                } else {
                    if (!planned) {
                        if (p.pull_bytes && (int)blockIdx.x >= p.head_units) {
                            // no head unit here: this CTA would only wait.  A hint, in 16 KB pieces dealt out over
                            // these CTAs; nothing depends on it.
                            const unsigned nb = gridDim.x - p.head_units, me = blockIdx.x - p.head_units;
                            const unsigned long long chunk = 16384, nchunks = (p.pull_bytes + chunk - 1) / chunk;
                            for (unsigned long long ch = me; ch < nchunks; ch += nb) {
                                const unsigned long long off = ch * chunk;
                                const unsigned sz = (unsigned)min(chunk, p.pull_bytes - off) & ~15u;
                                if (sz) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"((const char*)p.pull_ptr + off), "r"(sz) : "memory");
                            }
                        }
                        pdl_wait();
                        pdl_launch_dependents();
                        nu = *p.n_units - p.head_units;          // the list's head has been run
                        nsh = 0;
                        planned = true;
                    }
                    const unsigned long long old = atomicAdd(p.counter, 1ull);
                    u = (int)(uint32_t)old;
                    good = (unsigned long long)(uint32_t)old + (old >> 32) < (unsigned long long)nu;
                }
                if (good) {
                    // The list holds the shared expert's units first.  They are fed from L2 (every token tile of the
                    // model reads the same weights) while the routed units stream theirs from HBM, so the two kinds are
                    // dealt out alternately, in proportion: HBM then stays busy for the whole launch.
                    // The last sixth of the launch is kept for routed units: the shared ones are full-length, and a
                    // long unit handed out at the very end is what the other CTAs then wait for.
                    // (the short units at the tail of the list are taken in list order)
                    int ix = u;
                    const int n_main = nu - n_short;
                    if (nsh > 0 && u < n_main) {
                        const int routed = n_main - nsh;
                        const int cut = n_main - min(routed, n_main / 6);
                        const int uc = min(u, cut), uc1 = min(u + 1, cut);
                        const int a = (int)((long long)uc * nsh / cut), b = (int)((long long)uc1 * nsh / cut);
                        ix = b > a ? a : nsh + (u - a);
                    }
                    if (head) ix += p.head_units;
                    const Unit un = p.units[ix];
                    const Tile t = un.tile < 0 ? p.stiles[~un.tile] : p.tiles[un.tile];
                    e0 = make_int4(u, t.slot, t.row0, t.nrows);
                    e1 = make_int2(un.colblock & 0xffffff, un.tile < 0 ? 1 : 0);
                    e0w = 256 >> (un.colblock >> 24);
                } else if (from_plan) {
                    u = -1;
                }
                *reinterpret_cast<int4*>(&s_queue[q]) = e0;
                *reinterpret_cast<int2*>(&s_queue[q].colblock) = e1;
                s_queue[q].pad0 = e0w;
                s_queue[q].pad1 = from_plan;
                mbar_arrive(bar_qfull + 8 * q);
                if (PAIR) {
                    const uint32_t dst = peer_queue + (uint32_t)sizeof(QEntry) * q;
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(e0.x), "r"(e0.y), "r"(e0.z),
                                 "r"(e0.w) : "memory");
                    asm volatile("st.shared::cluster.v2.b32 [%0], {%1, %2};" ::"r"(dst + 16), "r"(e1.x), "r"(e1.y) : "memory");
                    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(dst + 24), "r"(e0w) : "memory");
                    mbar_arrive_cluster(peer_qfull + 8 * q);
                }
                if (++q == kQueue) { q = 0; qphase ^= 1; }
                if (u < 0) break;
            }
        }
        __syncwarp();
    } else if (BG) {
        bg_roles<MODE>(p, maps, warp, lane, rank, bg_ring, bg_full, bg_empty, bg_tfull, bg_tempty, bg_qfull, bg_qempty,
                       s_bg_queue, tmem_base, n_units, n_short, &s_abort);
    }

    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();      // nobody leaves while the peer may still read this CTA's memory or signal it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

__global__ void bf16_to_fp16_kernel(const bf16* __restrict__ src, __half* __restrict__ dst, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __float2half_rn(__bfloat162float(src[i]));
}

// 3-D map over two weight arrays of `rows` x `k` bf16 each: dimension 1 selects the array, so a box of
// (64 K, 2, 64 rows) lands in shared memory as 128 rows that alternate between the two arrays.
// Returns false on failure; *first_is_a tells whether index 0 of dimension 1 is array `a`.
bool make_pair_map(CUtensorMap* m, const void* a, const void* b, uint64_t rows, uint64_t k, uint32_t box_rows, bool* first_is_a)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const uintptr_t pa = (uintptr_t)a, pb = (uintptr_t)b;
    const uintptr_t lo = pa < pb ? pa : pb, hi = pa < pb ? pb : pa;
    *first_is_a = pa <= pb;
    const uint64_t diff = hi - lo;
    if (diff == 0 || (diff & 15) || diff >= (1ull << 40)) return false;
    cuuint64_t dims[3] = {k, 2, rows};
    cuuint64_t strides[2] = {diff, k * 2};
    cuuint32_t box[3] = {(cuuint32_t)kBK, 2, box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void*)lo, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct LayerMaps {
    bool ready = false;
    GemmMaps m1, m2;                    // weight maps of the gate/up and down GEMMs (activation maps are per call)
    GemmMaps m1t, m2t;                  // the same for the token-major shape (boxes of 256 / 128 / 64 weight rows)
    uint32_t gate_first_routed = 1, gate_first_shared = 0;
    std::vector<__half*> ws_down_f16;   // per model
};

struct TensorMaps {
    std::vector<LayerMaps> layers;
    int max_clusters[2] = {-1, -1};     // co-resident 2-CTA clusters of the pair kernels (without / with background lanes)
};

bool tc_supported(const moe_ctx* c)
{
    const moe_config& g = c->cfg;
    return g.hidden % 256 == 0 && g.inter % 128 == 0 && g.shared_inter % 128 == 0 && g.n_models <= kTcMaxModels;
}

// Long tiles: share the token tile between two CTAs.  The decision uses only host-side sizes.
bool tc_pair_mode(const moe_ctx* c, int T)
{
    const moe_config& g = c->cfg;
    (void)g;
    // measured (with 512-row tiles, two K slices per stage for the short units and the shared units dealt out between
    // the routed ones): the pair shape wins for every batch above 64 tokens -- prefill, the 240-expert pool with ~34
    // rows per expert, the 24-block stack, 96..2048 tokens of one model.  Up to 64 tokens the token-major shape, which
    // reads the tokens in place and needs no permuted copy, is faster (189.8 against 196.9 us at 32 tokens).
    if (c->pair_mode_enabled == 2) return true;        // (for measurements: the pair shape whatever the batch size)
    return c->pair_mode_enabled != 0 && T > 64;
}

// Tiles of up to 512 rows: the weight tile of a K step feeds two accumulators, so a CTA fetches 48 KB instead of
// 64 KB per 512 tokens; the 48 KB stages also let a short unit put two K slices into a stage.  The price is a
// shallower pipeline (4 stages) and, for full tiles, an epilogue that is not hidden behind the next unit.
bool tc_wide_mode(const moe_ctx* c, int T)
{
    return tc_pair_mode(c, T) && c->wide_tiles_enabled != 0;
}

// Pair shape: the short tiles (at most kShortRows rows) are run by a second, small pipeline of the same CTAs beside
// the long ones.
bool tc_background_mode(const moe_ctx* c, int T)
{
    // measured: it pays where long, tensor-bound tiles dominate and the short tiles can hide behind them (4096-token
    // prefill: step -3 %); where nearly every tile is short the launch is bound by HBM and the background lanes, with
    // their shallow ring, stream worse than the main ones (240-expert pool +8 %, 1126 tokens +6 %).  In between
    // (Zipf-skewed batches, rounds of 0.6 s alternating in one context): 2048 tokens +3 %, 2560 +1.4 %, 3072 +0.8 %,
    // 3584 +2 %, 4096 tokens -0.2 % on one part and -6.6 % on another.
    if (!tc_wide_mode(c, T) || c->background_enabled == 0) return false;
    return c->background_enabled == 2 || (c->cfg.n_models == 1 && T >= 4096);
}

// One-CTA units with the tokens as the M operand: every batch that does not take the pair shape.
bool tc_token_major(const moe_ctx* c, int T)
{
    return !tc_pair_mode(c, T) && c->token_major_enabled != 0;
}

void tc_destroy(moe_ctx* c)
{
    if (!c->tmaps) return;
    cudaDeviceSynchronize();
    for (LayerMaps& lm : c->tmaps->layers)
        for (__half* p : lm.ws_down_f16) if (p) cudaFree(p);
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
    memset(&lm.m1, 0, sizeof(GemmMaps));
    memset(&lm.m2, 0, sizeof(GemmMaps));
    memset(&lm.m1t, 0, sizeof(GemmMaps));
    memset(&lm.m2t, 0, sizeof(GemmMaps));
    bool ok = true, first = true;
    const uint64_t S = g.n_slots;
    ok &= make_pair_map(&lm.m1.a_routed[0], pw.w_gate, pw.w_up, S * I, H, 64, &first);
    lm.gate_first_routed = first ? 1u : 0u;
    ok &= make_map(&lm.m2.a_routed[0], pw.w_down, S * H, I, 128, false);
    for (int w = 0; w < 3; ++w) {       // token-major shape: 256, 128 and 64 weight rows per box
        ok &= make_pair_map(&lm.m1t.a_routed[w], pw.w_gate, pw.w_up, S * I, H, 128u >> w, &first);
        ok &= make_map(&lm.m2t.a_routed[w], pw.w_down, S * H, I, 256u >> w, false);
    }
    lm.ws_down_f16.assign(M, nullptr);
    lm.gate_first_shared = 0;
    for (int m = 0; m < M && ok && Is > 0; ++m) {
        const ModelWeights& mw = c->models[(size_t)layer * M + m];
        ok &= make_pair_map(&lm.m1.a_shared[m][0], mw.ws_gate, mw.ws_up, Is, H, 64, &first);
        for (int w = 0; w < 3; ++w) ok &= make_pair_map(&lm.m1t.a_shared[m][w], mw.ws_gate, mw.ws_up, Is, H, 128u >> w, &first);
        if (first) lm.gate_first_shared |= 1u << m;
        // fp16 copy of the shared expert's down projection (its activations are fp16 and one MMA takes
        // operands of one type); every bf16 weight of magnitude >= 2^-17 converts exactly
        const size_t n = (size_t)H * Is;
        if (cudaMalloc((void**)&lm.ws_down_f16[m], n * sizeof(__half)) != cudaSuccess) return MOE_ERR_ALLOC;
        bf16_to_fp16_kernel<<<(unsigned)((n + 255) / 256), 256>>>(mw.ws_down, lm.ws_down_f16[m], n);
        ok &= make_map(&lm.m2.a_shared[m][0], lm.ws_down_f16[m], H, Is, 128, true);
        for (int w = 0; w < 3; ++w) ok &= make_map(&lm.m2t.a_shared[m][w], lm.ws_down_f16[m], H, Is, 256u >> w, true);
    }
    if (!ok) {
        snprintf(c->errbuf, sizeof(c->errbuf), "cuTensorMapEncodeTiled failed for a weight tensor");
        return MOE_ERR_CUDA;
    }
    if (cudaDeviceSynchronize() != cudaSuccess) return MOE_ERR_CUDA;
    lm.ready = true;
    return MOE_OK;
}

namespace {

template <int MODE, bool PAIR, bool SWAP, bool BG>
cudaError_t launch_gemm(moe_ctx* c, const GemmParams& p, const GemmMaps& maps, cudaStream_t st, int grid_cap)
{
    auto kern = grouped_gemm_kernel<MODE, PAIR, SWAP, BG>;
    constexpr int kThr = BG ? kThreadsBg : kThreads;
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static bool attr_set[kMaxDevices] = {false};
    if (c->device < 0 || c->device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!attr_set[c->device]) {
        const cudaError_t ea = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (ea != cudaSuccess) return ea;
        attr_set[c->device] = true;
    }
    if (!PAIR) {
        return launch_pdl(kern, dim3(std::max(1, std::min(c->sm_count, grid_cap))), dim3(kThr), kSmemBytes, st, p, maps);
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.blockDim = dim3(kThr);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    int& max_clusters = c->tmaps->max_clusters[BG ? 1 : 0];
    if (max_clusters < 0) {
        // a persistent kernel must not launch more clusters than can be resident at once
        cfg.gridDim = dim3((unsigned)(c->sm_count & ~1));
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) n = 1;
        if (n > c->sm_count / 2) n = c->sm_count / 2;
        max_clusters = n;
    }
    cfg.gridDim = dim3((unsigned)(2 * std::max(1, std::min(max_clusters, grid_cap / 2))));
    return cudaLaunchKernelEx(&cfg, kern, p, maps);
}

}  // namespace

cudaError_t launch_experts_tc(moe_ctx* c, int layer, const bf16* x_or_xs, const bf16* x_perm, const int32_t* perm, int T,
                              float* y_perm, float* y_shared, const int32_t* shared_dst_rows, cudaStream_t st,
                              bool shared_only, bool tokens_ready)
{
    const moe_config& g = c->cfg;
    LayerMaps& lm = c->tmaps->layers[layer];
    const int H = g.hidden, I = g.inter, Is = g.shared_inter;
    const uint64_t R = (uint64_t)T * g.top_k;
    const bool shared = y_shared != nullptr && Is > 0;
    const bool pair = tc_pair_mode(c, T);
    const bool swap = tc_token_major(c, T);
    // direct mode: with few tokens the routed gate/up units read the tokens in place (no permuted copy)
    const bool direct = tc_direct_mode(c, T) && perm != nullptr && !shared_only;
    const uint32_t fmt_bf16 = (1u << 7) | (1u << 10), fmt_fp16 = 0u;

    // activation maps are rebuilt per call: their addresses and row counts are the call's
    GemmMaps& m1 = swap ? lm.m1t : lm.m1;
    bool ok = true;
    auto make_b = [](CUtensorMap* m, const void* base, uint64_t rows, uint64_t k, bool fp16) {
        bool good = true;
        for (int bx = 0; bx < 4; ++bx) good = good && make_map(m + bx, base, rows, k, 128u >> bx, fp16);
        return good && make_map(m + 4, base, rows, k, kBgAccRows / 2, fp16);
    };
    auto copy_b = [](CUtensorMap* dst, const CUtensorMap* src) { for (int bx = 0; bx < 5; ++bx) dst[bx] = src[bx]; };
    if (!direct && !shared_only) ok = make_b(m1.b_routed, x_perm, R, H, false);
    if (shared || direct) {
        ok = ok && make_b(m1.b_shared, x_or_xs, T, H, false);
        if (direct || shared_only) copy_b(m1.b_routed, m1.b_shared);
    } else {
        copy_b(m1.b_shared, m1.b_routed);
    }
    if (!ok) return cudaErrorInvalidValue;

    GemmParams p1;
    memset(&p1, 0, sizeof(p1));
    // the shared expert alone runs from unit lists of its own (it may be in flight beside the routed launches)
    int32_t* counts = shared_only ? c->ws.plan_counts_sh : c->ws.plan_counts;
    p1.units = shared_only ? c->ws.units1_sh : c->ws.units1;
    p1.n_units = counts + 2; p1.counter = reinterpret_cast<unsigned long long*>(counts + 10); p1.n_shared = counts + 6;
    p1.n_short = counts + 8;
    p1.tiles = c->ws.tiles; p1.stiles = shared_only ? c->ws.stiles_sh : c->ws.stiles;
    int cap1 = c->sm_count, cap2 = c->sm_count;
    if (shared_only) {
        // its unit counts are known on the host; a CTA pair shape leaves some SMs to the kernels it runs beside
        shared_unit_counts(c, T, &cap1, &cap2);
        if (pair) { cap1 = std::min(2 * cap1, c->early_shared_sms); cap2 = std::min(2 * cap2, c->early_shared_sms); }
    }
    p1.perm = perm; p1.top_k = g.top_k; p1.direct = direct ? 1 : 0; p1.n_tokens_pad = (T + 15) & ~15;
    p1.k_routed = H; p1.k_shared = H;
    p1.rows_per_slot = I; p1.cb_rows = swap ? 32 : 64;      // token-major: colblocks count steps of 64 weight rows
    p1.out_routed = c->ws.h; p1.out_shared = c->ws.hs; p1.ld_routed = I; p1.ld_shared = Is;
    p1.shared_dst_rows = nullptr;
    p1.idesc_fmt_routed = fmt_bf16; p1.idesc_fmt_shared = fmt_bf16;
    p1.gate_first_routed = lm.gate_first_routed; p1.gate_first_shared = lm.gate_first_shared;
    p1.status = c->ws.status;
    p1.stream_weights = (R <= 2048) ? 1 : 0;
    p1.wide = tc_wide_mode(c, T) ? 1 : 0;
    p1.group = p1.wide ? 1 : 2;
    if (swap) p1.group = 1;
    // Token-major shape, one model, all tokens in one tile: the shared expert's gate/up units need the tokens and static
    // weights only.  When the caller vouches that the tokens are final before the kernels ahead of this launch in the
    // stream began (a layer pass: router and dispatch only read them), the launch runs those units before it waits for
    // these kernels -- weight bytes streamed while the routing is still being worked out.
    if (tokens_ready && c->head_units_enabled && swap && shared && !shared_only && g.n_models == 1 && T <= kTileRows &&
        shared_dst_rows == nullptr) {
        p1.head_units = Is / 128;           // units of 256 interleaved gate / up rows
        p1.head_rows = T;
        // the CTAs beyond the head units fetch the shared expert's down weights (fp16 copy, 2 H Is bytes: they fit in L2
        // beside the head units' own tiles) for the launch that follows
        p1.pull_ptr = lm.ws_down_f16[0]; p1.pull_bytes = (unsigned long long)H * Is * 2;
    }
    // (the shared expert alone has no short tiles: its launches keep the shape without the background pipeline)
    const bool bg = pair && tc_background_mode(c, T) && !shared_only;
    cudaError_t e = pair ? (bg ? launch_gemm<0, true, false, true>(c, p1, m1, st, cap1)
                               : launch_gemm<0, true, false, false>(c, p1, m1, st, cap1))
                         : (swap ? launch_gemm<0, false, true, false>(c, p1, m1, st, cap1)
                                 : launch_gemm<0, false, false, false>(c, p1, m1, st, cap1));
    if (e != cudaSuccess) return e;
    if (!shared_only) stage_mark(c, st, kEvGateUp);

    GemmMaps& m2 = swap ? lm.m2t : lm.m2;
    ok = shared_only || make_b(m2.b_routed, c->ws.h, R, I, false);
    if (shared) ok = ok && make_b(m2.b_shared, c->ws.hs, T, Is, true);
    else copy_b(m2.b_shared, m2.b_routed);
    if (shared_only) copy_b(m2.b_routed, m2.b_shared);
    if (!ok) return cudaErrorInvalidValue;
    GemmParams p2 = p1;
    p2.head_units = 0; p2.head_rows = 0; p2.pull_bytes = 0;
    p2.units = shared_only ? c->ws.units2_sh : c->ws.units2;
    p2.n_units = counts + 3; p2.counter = reinterpret_cast<unsigned long long*>(counts + 12); p2.n_shared = counts + 7;
    p2.n_short = counts + 9;
    p2.direct = 0;
    p2.k_routed = I; p2.k_shared = Is;
    p2.rows_per_slot = H; p2.cb_rows = swap ? 64 : 128;
    p2.out_routed = y_perm; p2.out_shared = y_shared; p2.ld_routed = H; p2.ld_shared = H;
    p2.shared_dst_rows = shared_dst_rows;
    p2.idesc_fmt_routed = fmt_bf16; p2.idesc_fmt_shared = fmt_fp16;
    e = pair ? (bg ? launch_gemm<1, true, false, true>(c, p2, m2, st, cap2) : launch_gemm<1, true, false, false>(c, p2, m2, st, cap2))
             : (swap ? launch_gemm<1, false, true, false>(c, p2, m2, st, cap2)
                     : launch_gemm<1, false, false, false>(c, p2, m2, st, cap2));
    if (e != cudaSuccess) return e;
    if (!shared_only) stage_mark(c, st, kEvDown);
    c->launches += 2;
    return cudaGetLastError();
}

}  // namespace faasmoe
