"""GPU parity: the C-ABI CUDA path against the fp64 CPU oracle, element by element on
seeded inputs, from small and reduced cases up to the full sizes the benchmark times."""
import numpy as np
import pytest
import torch

import oracle
from harness import GpuLayer, assert_close, bf16_to_f64, check_routing, compare_four_calls, oracle_layer
from paper_2604_26881_b200 import binding as B
from paper_2604_26881_b200 import workloads as W

pytestmark = pytest.mark.gpu

PATHS = [B.MOE_PATH_FMA, B.MOE_PATH_AUTO]


@pytest.fixture(scope="module")
def qwen_weights():
    return W.make_weights(W.WORKLOADS["prefill"], seed=0)


def run_and_compare(wl, wts, x, tenant, mot, G, path, max_tokens=None):
    g = GpuLayer(wl, [wts], max_tokens or x.shape[0], model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_EXPERT_PATH, path)
        B.moe_set_option(g.ctx, B.MOE_OPT_ROUTE_PATH, path)
        o = g.four_calls(x, tenant, G)
        ref = oracle_layer(wl, wts, x, tenant, mot, G, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
        compare_four_calls(o, ref, wl, x)
        # the fused entry point equals the four calls bit for bit, and is reproducible
        out1 = g.forward(x, tenant, G)
        out2 = g.forward(x, tenant, G)
        assert torch.equal(out1, o["out"]) and torch.equal(out1, out2)
        return o, ref
    finally:
        g.close()


@pytest.mark.parametrize("path", PATHS)
def test_tiny_config(path):
    wl = W.WORKLOADS["tiny"]
    wts = W.make_weights(wl, seed=0)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    run_and_compare(wl, wts, x, tenant, mot, wl.G, path)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("G", [1, 5, 12])
def test_small_multi_model_pool(path, G):
    # 3 tenant models, 5 tenants, shuffled slot table, router bias, shared expert, G not dividing E,
    # a row count that spans several dispatch chunks and row tiles with ragged tails
    wl = W.MoEWorkload("small-pool", T=333, H=256, E=12, I=128, k=3, Is=256, M=3, n_tenants=5, G=G,
                       zipf_bias=True, tenant_layout="uniform")
    wts = W.make_weights(wl, seed=3, shuffle_slots=True)
    x, tenant, mot = W.make_tokens(wl, seed=3)
    o, ref = run_and_compare(wl, wts, x, tenant, mot, G, path, max_tokens=400)
    assert ref.dispatch.n_invocations <= 3 * -(-12 // G)


@pytest.mark.parametrize("H", [128, 384, 640])
@pytest.mark.parametrize("M", [1, 2])
def test_router_stage_counts_of_the_two_mma_lanes(H, M):
    # the tensor-core router splits its K stages between two MMA lanes (even / odd) with an accumulator each:
    # hidden sizes that give one stage (one lane only), three and five stages (lanes with unequal shares), with the
    # shared gate's rows riding in the same MMA, one and two models, a ragged last token tile
    wl = W.MoEWorkload("router-lanes", T=300, H=H, E=12, I=128, k=3, Is=128, M=M, n_tenants=3, G=4,
                       zipf_bias=True, tenant_layout="uniform")
    wts = W.make_weights(wl, seed=31)
    x, tenant, mot = W.make_tokens(wl, seed=31)
    run_and_compare(wl, wts, x, tenant, mot, wl.G, B.MOE_PATH_AUTO)


@pytest.mark.parametrize("path", PATHS)
def test_decode_config(qwen_weights, path):
    wl = W.WORKLOADS["decode"]
    wts = dict(qwen_weights, router_bias=None)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    o, ref = run_and_compare(wl, wts, x, tenant, mot, wl.G, path)
    assert 30 <= o["active_experts"] <= 60


@pytest.mark.parametrize("T", [1, 5, 33, 64, 100, 128])
def test_small_batches_token_major_units(qwen_weights, T):
    # batch sizes around the switches of the token-major plan: the shared expert's down units are 64 weight rows
    # wide up to 32 tokens, 128 up to 64 tokens, 256 above; the last round of units is split in two while the tiles
    # have at most 64 rows; up to 128 tokens the routed gate/up units read the tokens in place
    wl = W.scaled(W.WORKLOADS["decode"], T=T)
    wts = dict(qwen_weights, router_bias=None)
    x, tenant, mot = W.make_tokens(wl, seed=11)
    run_and_compare(wl, wts, x, tenant, mot, wl.G, B.MOE_PATH_AUTO)


@pytest.mark.parametrize("T", [2048, 2600])
def test_pair_shape_at_another_layer_shape(T):
    # the 2-CTA shape (512-row tiles, short units with two K slices per stage, shared units dealt out between the
    # routed ones) away from the Qwen sizes: 8 K steps, skewed loads from an empty expert to several tiles, every
    # element against the oracle
    wl = W.MoEWorkload("pair-small", T=T, H=512, E=8, I=256, k=2, Is=512, M=1, n_tenants=3, G=3,
                       zipf_bias=True, tenant_layout="uniform")
    wts = W.make_weights(wl, seed=21)
    x, tenant, mot = W.make_tokens(wl, seed=21)
    run_and_compare(wl, wts, x, tenant, mot, wl.G, B.MOE_PATH_AUTO)


@pytest.mark.parametrize("path", PATHS)
def test_prefill_reduced(qwen_weights, path):
    # the prefill layer (Zipf-skewed router) on 300 tokens: every element against the oracle
    wl = W.scaled(W.WORKLOADS["prefill"], T=300)
    x, tenant, mot = W.make_tokens(wl, seed=1)
    run_and_compare(wl, qwen_weights, x, tenant, mot, wl.G, path)


def test_prefill_full_size_every_token(qwen_weights):
    # full 4096-token prefill in the launch configuration the benchmark times (fused entry point, shared expert on
    # the second stream), then the four calls at the same size: every output of every stage -- routing, tie flags,
    # permutation, offsets, un-weighted expert outputs of all 16,384 routed rows and 4,096 shared rows, layer output
    # -- against the oracle, element by element
    wl = W.WORKLOADS["prefill"]
    x, tenant, mot = W.make_tokens(wl, seed=0)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        out = g.forward(x, tenant, wl.G)
        status = B.moe_last_status(g.ctx)
        assert status[0] == 0
        o = g.four_calls(x, tenant, wl.G)
        assert torch.equal(out, o["out"])
        ref = oracle_layer(wl, qwen_weights, x, tenant, mot, wl.G, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
        compare_four_calls(o, ref, wl, x)
        assert status[1] == ref.dispatch.n_invocations
        # expert load is skewed as the workload asks
        load = np.diff(ref.dispatch.expert_off)
        assert load.max() > 8 * max(1, np.median(load))
    finally:
        g.close()


def test_qwen_shape_without_shared_expert(qwen_weights):
    # the routed path alone at the Qwen layer shape: with a shared expert its term is about three times the routed
    # one in the layer output, so the output tolerance is loose for the routed experts; here nothing hides them
    wl = W.scaled(W.WORKLOADS["prefill"], T=600, Is=0)
    wts = dict(qwen_weights, shared_gate_w=None, ws_gate=None, ws_up=None, ws_down=None)
    x, tenant, mot = W.make_tokens(wl, seed=8)
    for path in PATHS:
        run_and_compare(wl, wts, x, tenant, mot, wl.G, path)
    wl = W.scaled(W.WORKLOADS["decode"], Is=0)
    x, tenant, mot = W.make_tokens(wl, seed=8)
    run_and_compare(wl, dict(wts, router_bias=None), x, tenant, mot, wl.G, B.MOE_PATH_AUTO)


@pytest.mark.parametrize("path", PATHS)
def test_tie_flag_on_both_sides_of_the_threshold(path):
    # two experts with identical router rows and biases that differ by a chosen amount are ranks 1 and 2 of every
    # token with a relative probability gap of 1 - exp(-delta): below the 1e-5 threshold every token must be
    # flagged, above it the flag must equal the oracle's (which then depends on the other ranks only)
    wl = W.MoEWorkload("ties", T=200, H=256, E=12, I=128, k=3, Is=128, M=1, n_tenants=2, G=4, tenant_layout="uniform")
    base = W.make_weights(wl, seed=41)
    x, tenant, mot = W.make_tokens(wl, seed=41)
    for ulps, expect_all in ((6, True), (64, False)):
        wts = dict(base)
        rw = base["router_w"].clone()
        rw[0, 7] = rw[0, 2]
        bias = torch.zeros((1, wl.E), dtype=torch.float32)
        delta = ulps * 2.0 ** -21                 # float32 spacing in [4, 8) is 2^-21: 6 ulps = 2.9e-6, 64 ulps = 3.1e-5
        bias[0, 2], bias[0, 7] = 6.0, 6.0 - delta
        wts["router_w"], wts["router_bias"] = rw, bias
        g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
        try:
            B.moe_set_option(g.ctx, B.MOE_OPT_ROUTE_PATH, path)
            o = g.four_calls(x, tenant, wl.G)
            ref = oracle_layer(wl, wts, x, tenant, mot, wl.G, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
            compare_four_calls(o, ref, wl, x)         # includes the flag comparison on every decided token
            flag = o["tie_flag"].cpu().numpy().astype(bool)
            p = -np.sort(-ref.routing.probs, axis=1)
            gap01 = (p[:, 0] - p[:, 1]) / p[:, 0]
            assert np.all(np.sort(o["topk_idx"].cpu().numpy()[:, :2], axis=1) == [2, 7])
            if expect_all:
                assert gap01.max() < 0.5e-5 and flag.all() and ref.routing.tie_flag.all()
            else:
                assert gap01.min() > 2e-5
                assert np.array_equal(flag, ref.routing.tie_flag.astype(bool)) and not flag.all()
        finally:
            g.close()


@pytest.mark.parametrize("path", PATHS)
def test_pool_config_reduced_and_G_sweep(path):
    # 4 tenant models in one pool, top-4 inside each tenant's own experts, uniform tenant ids
    wl = W.scaled(W.WORKLOADS["pool"], T=192, H=512, I=256, Is=512, E=60)
    wts = W.make_weights(wl, seed=5, shuffle_slots=True)
    x, tenant, mot = W.make_tokens(wl, seed=5)
    o, ref = run_and_compare(wl, wts, x, tenant, mot, 1, path)
    g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_EXPERT_PATH, path)
        B.moe_set_option(g.ctx, B.MOE_OPT_ROUTE_PATH, path)
        base = g.forward(x, tenant, 1)
        assert torch.equal(base, o["out"])
        invocations = []
        for G in (1, 2, 4, 6, 12, 60):
            out = g.forward(x, tenant, G)
            assert torch.equal(out, base), f"output changed with G={G}"      # bit-identical for every G
            invocations.append(B.moe_last_status(g.ctx)[1])
        assert invocations == sorted(invocations, reverse=True) and invocations[-1] == 4
    finally:
        g.close()


@pytest.mark.parametrize("path", PATHS)
def test_stack_teacher_forced(path):
    # 3 blocks of RMSNorm -> MoE (+shared) -> residual; ragged multi-tenant batch
    wl = W.scaled(W.WORKLOADS["stack"], H=512, I=256, Is=512, E=24, n_layers=3, n_tenants=6)
    layers = [W.make_weights(wl, seed=7, layer=l) for l in range(wl.n_layers)]
    x, tenant, mot = W.make_tokens(wl, seed=7)
    x, tenant = x[:700].contiguous(), tenant[:700].contiguous()
    T = x.shape[0]
    g = GpuLayer(wl, layers, T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_EXPERT_PATH, path)
        B.moe_set_option(g.ctx, B.MOE_OPT_ROUTE_PATH, path)
        xd, td = x.to(g.dev).clone(), tenant.to(g.dev)
        dbg_in = torch.zeros((wl.n_layers, T, wl.H), dtype=torch.bfloat16, device=g.dev)
        dbg_out = torch.zeros_like(dbg_in)
        B.moe_stack_forward(g.ctx, xd, td, T, wl.G, dbg_in, dbg_out)
        torch.cuda.synchronize()
        assert B.moe_last_status(g.ctx)[0] == 0
        assert torch.equal(dbg_out[-1], xd)
        # teacher forcing: block l of the oracle starts from the GPU's residual stream and the GPU's
        # normalised input, so every block is compared on identical inputs
        x_in = x
        for l in range(wl.n_layers):
            wn = W.weights_as_numpy(layers[l])
            xn_ref = oracle.rmsnorm(W.as_u16(x_in), wn["rms_w"], wl.rms_eps)
            xn_gpu = dbg_in[l].cpu()
            ulp = 2.0 ** (np.floor(np.log2(np.abs(xn_ref) + 1e-300)) - 7)      # spacing of bf16 at each value
            err = np.abs(bf16_to_f64(xn_gpu) - xn_ref) / ulp
            assert err.max() <= 1.0, f"block {l}: RMSNorm differs by {err.max()} bf16 ulp"
            # the gate alone on the GPU's xn, to apply the near-tie protocol to this block
            tk_i = torch.zeros((T, wl.k), dtype=torch.int32, device=g.dev)
            tk_w = torch.zeros((T, wl.k), dtype=torch.float32, device=g.dev)
            B.moe_route(g.ctx, l, dbg_in[l], td, T, tk_i, tk_w)
            torch.cuda.synchronize()
            r = oracle.route(W.as_u16(xn_gpu), tenant.numpy(), mot.numpy(), wn["router_w"], wn["router_bias"],
                             wn["shared_gate_w"], k=wl.k)
            ov = check_routing(tk_i.cpu().numpy(), tk_w.cpu().numpy(), r, wl.k)
            _, _, res = oracle.block_forward(W.as_u16(x_in), tenant.numpy(), mot.numpy(), wn, k=wl.k, G=wl.G,
                                             eps=wl.rms_eps, xn_override=W.as_u16(xn_gpu), topk_override=ov)
            assert_close(f"block {l} residual stream", bf16_to_f64(dbg_out[l]), bf16_to_f64(x_in) + res.out)
            x_in = dbg_out[l].cpu()
        # the stack without debug buffers gives the same bits
        xd2 = x.to(g.dev).clone()
        B.moe_stack_forward(g.ctx, xd2, td, T, wl.G)
        torch.cuda.synchronize()
        assert torch.equal(xd2, xd)
    finally:
        g.close()


@pytest.mark.parametrize("T", [5, 40, 64])
def test_small_stack_agrees_across_wait_options(T):
    # a stack of four blocks on a decode-sized batch: in every block the gate/up launch may start on the shared
    # expert's units while the block's RMSNorm output is being routed, and the dispatch may run inside the router's
    # launch.  The block's input is the previous block's output, so a launch that ran ahead of data it needs would
    # show in the residual stream; all four settings must give the same bits, twice in a row.
    wl = W.scaled(W.WORKLOADS["stack"], H=512, I=256, Is=512, E=24, n_layers=4, n_tenants=6, T=T, tenant_layout="uniform")
    layers = [W.make_weights(wl, seed=11, layer=l) for l in range(wl.n_layers)]
    x, tenant, mot = W.make_tokens(wl, seed=11)
    g = GpuLayer(wl, layers, T, model_of_tenant=mot)
    try:
        td = tenant.to(g.dev)
        outs = {}
        for head in (0, 1):
            for fused in (0, 1):
                B.moe_set_option(g.ctx, B.MOE_OPT_HEAD_UNITS, head)
                B.moe_set_option(g.ctx, B.MOE_OPT_FUSED_DISPATCH, fused)
                runs = []
                for _ in range(2):
                    xd = x.to(g.dev).clone()
                    B.moe_stack_forward(g.ctx, xd, td, T, wl.G)
                    runs.append(xd)
                torch.cuda.synchronize()
                assert B.moe_last_status(g.ctx)[0] == 0
                assert torch.equal(runs[0], runs[1])
                outs[(head, fused)] = runs[0]
        ref = outs[(0, 0)]
        assert not torch.equal(ref, x.to(g.dev))
        for key, o in outs.items():
            assert torch.equal(o, ref), key
    finally:
        g.close()


def test_pair_shape_and_single_shape_agree_bit_for_bit(qwen_weights):
    # the 2-CTA (cta_group::2) and the 1-CTA shape of the grouped GEMM tile the work differently but
    # accumulate every output element over K in the same order
    wl = W.scaled(W.WORKLOADS["prefill"], T=1024)
    x, tenant, mot = W.make_tokens(wl, seed=2)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_PAIR_MODE, 2)
        pair = g.forward(x, tenant, wl.G)
        B.moe_set_option(g.ctx, B.MOE_OPT_PAIR_MODE, 0)
        single = g.forward(x, tenant, wl.G)              # one CTA per unit, tokens as the M operand
        B.moe_set_option(g.ctx, B.MOE_OPT_TOKEN_MAJOR, 0)
        single_wm = g.forward(x, tenant, wl.G)           # one CTA per unit, weight rows as the M operand
        assert B.moe_last_status(g.ctx)[0] == 0
        assert torch.equal(pair, single) and torch.equal(pair, single_wm)
        # and both are the CUDA-core path within the tolerance
        B.moe_set_option(g.ctx, B.MOE_OPT_EXPERT_PATH, B.MOE_PATH_FMA)
        fma = g.forward(x, tenant, wl.G)
        assert_close("pair vs fma", bf16_to_f64(pair), bf16_to_f64(fma))
    finally:
        g.close()


@pytest.mark.parametrize("T", [1024, 1500, 4096])
def test_wide_tiles_and_narrow_tiles_agree_bit_for_bit(qwen_weights, T):
    # tiles of up to 512 rows feed two accumulators from one weight tile; every output element is
    # still accumulated over K in the same order as with 256-row tiles.  The Zipf-skewed router
    # gives segments of every length: shorter than 256, between 256 and 512, and several tiles long.
    wl = W.scaled(W.WORKLOADS["prefill"], T=T)
    x, tenant, mot = W.make_tokens(wl, seed=4)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_WIDE_TILES, 2)
        wide = g.forward(x, tenant, wl.G)
        B.moe_set_option(g.ctx, B.MOE_OPT_WIDE_TILES, 0)
        narrow = g.forward(x, tenant, wl.G)
        assert B.moe_last_status(g.ctx)[0] == 0
        assert torch.equal(wide, narrow)
    finally:
        g.close()


@pytest.mark.parametrize("T", [200, 1500, 4096])
def test_background_lanes_agree_bit_for_bit(qwen_weights, T):
    # the 2-CTA shape may run the short tiles (at most 64 rows) in a second pipeline beside the long ones; which
    # pipeline runs a unit, and in what order, depends on timing, the result does not: every output element is summed
    # over K in the same order by one lane.  Several tenants and the private orchestrator mode give many short tiles;
    # calls back to back reuse the work counters.
    wl = W.scaled(W.WORKLOADS["prefill"], T=T, n_tenants=5, tenant_layout="uniform")
    x, tenant, mot = W.make_tokens(wl, seed=9)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        for mode in (B.MOE_DISPATCH_SHARED, B.MOE_DISPATCH_PRIVATE):
            B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, mode)
            for early in (0, 2):
                B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, early)
                B.moe_set_option(g.ctx, B.MOE_OPT_BACKGROUND_LANES, 0)
                ref = g.forward(x, tenant, wl.G)
                B.moe_set_option(g.ctx, B.MOE_OPT_BACKGROUND_LANES, 2)
                outs = [g.forward(x, tenant, wl.G) for _ in range(4)]
                assert B.moe_last_status(g.ctx)[0] == 0
                for o in outs:
                    assert torch.equal(o, ref), (mode, early)
        # and against the oracle through the four calls, background lanes on
        o = g.four_calls(x, tenant, wl.G)
        ref = oracle_layer(wl, qwen_weights, x, tenant, mot, wl.G, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
        o["n_invocations"] = ref.dispatch.n_invocations      # (private mode counts per tenant: checked elsewhere)
        compare_four_calls(o, ref, wl, x)
    finally:
        g.close()


@pytest.mark.parametrize("T", [1, 5, 32, 100, 128, 129])
def test_dispatch_behind_the_router_agrees_bit_for_bit(qwen_weights, T):
    # a batch that one CTA routes (at most 128 tokens of one model) is dispatched, and its experts' work laid out, by
    # that CTA in the router's launch; the same code runs as a launch of its own otherwise (129 tokens: always).
    # Outputs, routing buffers, offsets, statistics and the number of launches are compared, in both orchestrator
    # modes, with and without a block table, the batch changing from call to call.
    wl = W.scaled(W.WORKLOADS["decode"], T=T, n_tenants=3, tenant_layout="uniform")
    x, tenant, mot = W.make_tokens(wl, seed=21)
    x2, tenant2, _ = W.make_tokens(wl, seed=22)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    R = T * wl.k
    try:
        ws = B.moe_get_workspace(g.ctx)
        shapes = {"topk_idx": ((R,), torch.int32), "topk_w": ((R,), torch.float32), "shared_gate": ((T,), torch.float32),
                  "tie_flag": ((T,), torch.uint8), "perm": ((R,), torch.int32), "inv_perm": ((R,), torch.int32),
                  "expert_off": ((wl.E + 1,), torch.int32)}

        def run(fused, xx, tt, G):
            B.moe_set_option(g.ctx, B.MOE_OPT_FUSED_DISPATCH, fused)
            n0 = B.moe_launch_count(g.ctx)
            out = g.forward(xx, tt, G)
            n = B.moe_launch_count(g.ctx) - n0
            bufs = {k: B.wrap_device_pointer(ws[k], sh, dt, g.dev).clone() for k, (sh, dt) in shapes.items()}
            return out, bufs, B.moe_last_status(g.ctx), B.moe_last_plan(g.ctx, T), n

        for mode in (B.MOE_DISPATCH_SHARED, B.MOE_DISPATCH_PRIVATE):
            B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, mode)
            for table in (False, True):
                if table:
                    B.moe_set_block_table(g.ctx, torch.tensor([[(7 * e + 3) % 9 for e in range(wl.E)]], dtype=torch.int32), 9)
                else:
                    B.moe_set_block_table(g.ctx, None)
                for G in (1, 4):
                    for xx, tt in ((x, tenant), (x2, tenant2)):
                        ref = run(0, xx, tt, G)
                        got = run(1, xx, tt, G)
                        assert got[2][0] == 0 and ref[2][0] == 0
                        assert torch.equal(got[0], ref[0]), (mode, table, G)
                        for k in shapes:
                            assert torch.equal(got[1][k], ref[1][k]), (k, mode, table, G)
                        assert got[2] == ref[2] and got[3] == ref[3]
                        assert got[4] == ref[4] - (1 if T <= 128 else 0)
    finally:
        g.close()


@pytest.mark.parametrize("T", [1, 8, 32, 64])
def test_shared_units_ahead_of_the_wait_agree_bit_for_bit(qwen_weights, T):
    # small batches of one model: the gate/up launch may run the shared expert's units (tokens and static weights only)
    # before it waits for the router and the dispatch of the same pass.  Same units, same arithmetic: the output bits
    # do not change, with the dispatch inside the router's launch or in its own, call after call without a
    # synchronisation in between (the launch of one pass starts while kernels of the pass before may still run) and
    # with the batch changing from call to call.
    wl = W.scaled(W.WORKLOADS["decode"], T=T, n_tenants=3, tenant_layout="uniform")
    x, tenant, mot = W.make_tokens(wl, seed=31)
    x2, tenant2, _ = W.make_tokens(wl, seed=32)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_HEAD_UNITS, 0)
        ref, ref2 = g.forward(x, tenant, wl.G), g.forward(x2, tenant2, wl.G)
        xd, td, xd2, td2 = x.to(g.dev), tenant.to(g.dev), x2.to(g.dev), tenant2.to(g.dev)
        for fused in (1, 0):
            B.moe_set_option(g.ctx, B.MOE_OPT_FUSED_DISPATCH, fused)
            B.moe_set_option(g.ctx, B.MOE_OPT_HEAD_UNITS, 1)
            outs = [torch.zeros_like(xd) for _ in range(8)]
            for i, o in enumerate(outs):
                B.moe_layer_forward(g.ctx, 0, xd if i % 2 == 0 else xd2, td if i % 2 == 0 else td2, T, wl.G, o)
            torch.cuda.synchronize()
            assert B.moe_last_status(g.ctx)[0] == 0
            for i, o in enumerate(outs):
                assert torch.equal(o, ref if i % 2 == 0 else ref2), (fused, i)
        # and against the oracle, element by element, through the fused entry point
        o = g.four_calls(x, tenant, wl.G)
        want = oracle_layer(wl, qwen_weights, x, tenant, mot, wl.G, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
        compare_four_calls(o, want, wl, x)
        assert torch.equal(ref, o["out"])
    finally:
        g.close()


@pytest.mark.parametrize("T", [7, 64, 300, 1024, 4096])
def test_shared_expert_on_second_stream_agrees_bit_for_bit(qwen_weights, T):
    # one model: the shared expert's launches may run on the context's second stream beside the router and the
    # dispatch.  The same units do the same arithmetic, so the output bits do not change, call after call (the
    # buffers of one call are reused by the next one while two streams are in flight).
    wl = W.scaled(W.WORKLOADS["prefill"], T=T)
    x, tenant, mot = W.make_tokens(wl, seed=6)
    x2, tenant2, _ = W.make_tokens(wl, seed=7)
    g = GpuLayer(wl, [qwen_weights], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 0)
        ref, ref2 = g.forward(x, tenant, wl.G), g.forward(x2, tenant2, wl.G)
        for sms in (116, 32, 148):
            B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 2)
            B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED_SMS, sms)
            xd, td, xd2, td2 = x.to(g.dev), tenant.to(g.dev), x2.to(g.dev), tenant2.to(g.dev)
            outs = [torch.zeros_like(xd) for _ in range(6)]
            for i, o in enumerate(outs):                 # back to back, no synchronisation in between
                B.moe_layer_forward(g.ctx, 0, xd if i % 2 == 0 else xd2, td if i % 2 == 0 else td2, T, wl.G, o)
            torch.cuda.synchronize()
            assert B.moe_last_status(g.ctx)[0] == 0
            for i, o in enumerate(outs):
                assert torch.equal(o, ref if i % 2 == 0 else ref2), (sms, i)
    finally:
        g.close()


def test_token_grouping_on_second_stream_agrees_bit_for_bit():
    # several models: the tokens are grouped by model (input of the shared experts) on the context's second stream
    # while the router and the dispatch run; calls back to back reuse the grouping buffers
    wl = W.MoEWorkload("small-pool", T=333, H=256, E=12, I=128, k=3, Is=256, M=3, n_tenants=5, G=5,
                       zipf_bias=True, tenant_layout="uniform")
    wts = W.make_weights(wl, seed=3, shuffle_slots=True)
    x, tenant, mot = W.make_tokens(wl, seed=3)
    x2, tenant2, _ = W.make_tokens(wl, seed=4)
    g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    try:
        B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 0)
        ref, ref2 = g.forward(x, tenant, wl.G), g.forward(x2, tenant2, wl.G)
        B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 1)
        xd, td, xd2, td2 = x.to(g.dev), tenant.to(g.dev), x2.to(g.dev), tenant2.to(g.dev)
        outs = [torch.zeros_like(xd) for _ in range(6)]
        for i, o in enumerate(outs):
            B.moe_layer_forward(g.ctx, 0, xd if i % 2 == 0 else xd2, td if i % 2 == 0 else td2, wl.T, wl.G, o)
        torch.cuda.synchronize()
        assert B.moe_last_status(g.ctx)[0] == 0
        for i, o in enumerate(outs):
            assert torch.equal(o, ref if i % 2 == 0 else ref2), i
    finally:
        g.close()


@pytest.mark.parametrize("seed", [6, 7])
def test_random_small_configurations_against_the_oracle(seed):
    # 30 random small layer shapes per seed, every output of the four calls against the oracle element by element:
    # hidden sizes with one to six K stages of the router (H = 128 ... 768; the experts run on the CUDA cores where
    # H is not a multiple of 256), E = 3 ... 64, top-1 ... top-6, one to four models (a router CTA per model), with and
    # without a shared expert, block sizes that do not divide E, 1 ... 400 tokens
    import random
    rng = random.Random(seed)
    for it in range(30):
        H = rng.choice([128, 256, 384, 512, 640, 768]); E = rng.choice([3, 8, 12, 16, 33, 60, 64])
        I = rng.choice([128, 256]); k = rng.randint(1, min(6, E))
        Is = rng.choice([0, 128, 256]); M = rng.choice([1, 2, 3, 4]); nt = rng.randint(M, M + 3)
        G = rng.randint(1, E)
        T = rng.choice([1, 5, 31, 64, 65, 130, 257, 400])
        wl = W.MoEWorkload(f"random{it}", T=T, H=H, E=E, I=I, k=k, Is=Is, M=M, n_tenants=nt, G=G,
                           zipf_bias=rng.random() < 0.5, tenant_layout=rng.choice(["uniform", "contiguous"]))
        wts = W.make_weights(wl, seed=100 + it, shuffle_slots=rng.random() < 0.5)
        x, tenant, mot = W.make_tokens(wl, seed=100 + it)
        run_and_compare(wl, wts, x, tenant, mot, G, B.MOE_PATH_AUTO)


@pytest.mark.parametrize("seed", [2, 3])
def test_random_configurations_agree_across_entry_points_and_paths(seed):
    # 20 random layer shapes per seed (hidden size, experts, top-k, shared expert or none, one to four models, block
    # size, 1 ... 4096 tokens): the fused entry point equals the four calls bit for bit, with the shared expert on the
    # second stream or not, is reproducible, and stays within the tolerance of the CUDA-core expert path
    import random
    rng = random.Random(seed)
    for it in range(20):
        H = rng.choice([256, 512, 768, 1024, 2048]); E = rng.choice([4, 8, 12, 16, 33, 60, 64])
        I = rng.choice([128, 256, 384]); k = rng.randint(1, min(6, E))
        Is = rng.choice([0, 128, 256, 512]); M = rng.choice([1, 1, 2, 3, 4]); nt = rng.randint(M, M + 4)
        G = rng.randint(1, E)
        T = rng.choice([1, 2, 3, 17, 31, 64, 65, 100, 128, 129, 255, 300, 513, 700, 1025, 1500, 2600, 4096])
        wl = W.MoEWorkload(f"random{it}", T=T, H=H, E=E, I=I, k=k, Is=Is, M=M, n_tenants=nt, G=G,
                           zipf_bias=rng.random() < 0.5, tenant_layout=rng.choice(["uniform", "contiguous"]))
        wts = W.make_weights(wl, seed=it, shuffle_slots=rng.random() < 0.5)
        x, tenant, mot = W.make_tokens(wl, seed=it)
        g = GpuLayer(wl, [wts], T, model_of_tenant=mot)
        try:
            o = g.four_calls(x, tenant, G)
            f1, f2 = g.forward(x, tenant, G), g.forward(x, tenant, G)
            B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 2)
            f3 = g.forward(x, tenant, G)
            B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, 0)
            f4 = g.forward(x, tenant, G)
            assert B.moe_last_status(g.ctx)[0] == 0, wl
            assert torch.equal(f1, o["out"]) and torch.equal(f1, f2) and torch.equal(f1, f3) and torch.equal(f1, f4), wl
            B.moe_set_option(g.ctx, B.MOE_OPT_EXPERT_PATH, B.MOE_PATH_FMA)
            fma = g.forward(x, tenant, G)
            assert_close(f"{wl}: tensor-core vs CUDA-core experts", bf16_to_f64(f1), bf16_to_f64(fma))
        finally:
            g.close()


def test_pool_full_size_G_sweep_every_token():
    # 4 tenant models, 240 routed slots + 4 shared experts in one pool (4.4 GB), 2048 tokens with uniform
    # tenant ids, shuffled slot table: outputs bit-identical for every G; every output of the four calls (all 8,192
    # routed rows, all tokens) against the oracle
    wl = W.WORKLOADS["pool"]
    wts = W.make_weights(wl, seed=0, shuffle_slots=True)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    try:
        base = g.forward(x, tenant, 1)
        o = g.four_calls(x, tenant, 1)
        assert torch.equal(base, o["out"])
        ref = oracle_layer(wl, wts, x, tenant, mot, 1, o["topk_idx"].cpu().numpy(), o["topk_w"].cpu().numpy())
        compare_four_calls(o, ref, wl, x)
        inv = []
        for G in (1, 2, 4, 6, 12, 60):
            out = g.forward(x, tenant, G)
            st = B.moe_last_status(g.ctx)
            assert st[0] == 0 and torch.equal(out, base), f"G={G}"
            inv.append(st[1])
        assert inv[0] == st[2] and inv[-1] == 4 and inv == sorted(inv, reverse=True)
    finally:
        g.close()


def test_stack_full_size_teacher_forced():
    # 24 blocks, 26.6 GB of weights resident, 16 tenants with ragged request lengths, G = 6.  Blocks 0, 11
    # and 23 have CPU twins of their weights and are checked against the oracle from the GPU's own block
    # inputs, on every token; the other blocks get device-generated weights of the same distribution.
    wl = W.WORKLOADS["stack"]
    if torch.cuda.mem_get_info()[0] < 40e9:
        pytest.skip("needs about 30 GB of free device memory")
    x, tenant, mot = W.make_tokens(wl, seed=0)
    T = x.shape[0]
    checked = {0: None, 11: None, 23: None}
    dev = torch.device("cuda:0")
    layers = []
    gen = torch.Generator(device=dev).manual_seed(1234)
    for l in range(wl.n_layers):
        if l in checked:
            checked[l] = W.make_weights(wl, seed=0, layer=l)
            layers.append(checked[l])
        else:
            def rnd(*shape, std=0.02):
                return (torch.randn(*shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
            S = wl.n_slots
            layers.append({
                "router_w": rnd(1, wl.E, wl.H), "router_bias": None,
                "pool_gate": rnd(S, wl.I, wl.H), "pool_up": rnd(S, wl.I, wl.H), "pool_down": rnd(S, wl.H, wl.I),
                "shared_gate_w": rnd(1, wl.H), "ws_gate": rnd(1, wl.Is, wl.H), "ws_up": rnd(1, wl.Is, wl.H),
                "ws_down": rnd(1, wl.H, wl.Is), "slot_table": torch.arange(S, dtype=torch.int32),
                "rms_w": (1.0 + torch.randn(wl.H, generator=gen, device=dev) * 0.02).to(torch.bfloat16)})
    g = GpuLayer(wl, layers, T, model_of_tenant=mot)
    try:
        xd, td = x.to(dev).clone(), tenant.to(dev)
        dbg_in = torch.zeros((wl.n_layers, T, wl.H), dtype=torch.bfloat16, device=dev)
        dbg_out = torch.zeros_like(dbg_in)
        B.moe_stack_forward(g.ctx, xd, td, T, wl.G, dbg_in, dbg_out)
        torch.cuda.synchronize()
        assert B.moe_last_status(g.ctx)[0] == 0
        assert torch.isfinite(xd.float()).all()
        for l, wts in checked.items():
            wn = W.weights_as_numpy(wts)
            x_in = (x if l == 0 else dbg_out[l - 1].cpu())
            xn_gpu = dbg_in[l].cpu()
            xn_ref = oracle.rmsnorm(W.as_u16(x_in), wn["rms_w"], wl.rms_eps)
            ulp = 2.0 ** (np.floor(np.log2(np.abs(xn_ref) + 1e-300)) - 7)
            assert (np.abs(bf16_to_f64(xn_gpu) - xn_ref) / ulp).max() <= 1.0
            tk_i = torch.zeros((T, wl.k), dtype=torch.int32, device=dev)
            tk_w = torch.zeros((T, wl.k), dtype=torch.float32, device=dev)
            B.moe_route(g.ctx, l, dbg_in[l], td, T, tk_i, tk_w)
            torch.cuda.synchronize()
            r = oracle.route(W.as_u16(xn_gpu), tenant.numpy(), mot.numpy(), wn["router_w"], wn["router_bias"],
                             wn["shared_gate_w"], k=wl.k)
            ov = check_routing(tk_i.cpu().numpy(), tk_w.cpu().numpy(), r, wl.k)
            _, _, res = oracle.block_forward(W.as_u16(x_in), tenant.numpy(), mot.numpy(), wn, k=wl.k, G=wl.G, eps=wl.rms_eps,
                                             xn_override=W.as_u16(xn_gpu), topk_override=ov)
            assert_close(f"block {l} residual stream", bf16_to_f64(dbg_out[l]), bf16_to_f64(x_in) + res.out)
    finally:
        g.close()


@pytest.mark.parametrize("seed", [4, 5, 6])
def test_random_configurations_agree_across_modes_tables_and_lanes(seed):
    # 25 random layer shapes per seed, four random option settings each -- shared or private orchestrators, blocks by
    # ranges or by a load-aware table, background lanes off or forced on, the shared expert on the second stream or not:
    # none of them may change a bit of the output or leave a device status bit.  Seed 6 draws small batches (at most
    # 128 tokens) and also switches the shared expert's units ahead of the wait and the dispatch inside the router's
    # launch on and off (the reference run has both off).
    import random
    rng = random.Random(seed)
    for it in range(25):
        H = rng.choice([256, 512, 1024, 2048]); E = rng.choice([4, 8, 12, 16, 33, 60, 64])
        I = rng.choice([128, 256, 384]); k = rng.randint(1, min(6, E))
        Is = rng.choice([0, 128, 256, 512]); M = rng.choice([1, 1, 1, 2, 3]); nt = rng.randint(M, M + 5)
        G = rng.randint(1, E)
        T = rng.choice([1, 3, 31, 64, 65, 100, 128, 129, 255, 300, 513, 700, 1025, 1500, 2048, 2600, 4096])
        if seed >= 6:
            T = rng.choice([1, 2, 3, 8, 17, 31, 32, 48, 63, 64, 65, 100, 128])
        wl = W.MoEWorkload(f"random{it}", T=T, H=H, E=E, I=I, k=k, Is=Is, M=M, n_tenants=nt, G=G,
                           zipf_bias=rng.random() < 0.6, tenant_layout=rng.choice(["uniform", "contiguous"]))
        wts = W.make_weights(wl, seed=500 + it, shuffle_slots=rng.random() < 0.5)
        x, tenant, mot = W.make_tokens(wl, seed=500 + it)
        g = GpuLayer(wl, [wts], T, model_of_tenant=mot)
        try:
            if seed >= 6:
                B.moe_set_option(g.ctx, B.MOE_OPT_HEAD_UNITS, 0)
                B.moe_set_option(g.ctx, B.MOE_OPT_FUSED_DISPATCH, 0)
            base = g.forward(x, tenant, G)
            ws = B.moe_get_workspace(g.ctx)
            eoff = B.wrap_device_pointer(ws["expert_off"], (M * E + 1,), torch.int32, g.dev).cpu().to(torch.int64)
            table = B.moe_form_blocks((eoff[1:] - eoff[:-1]).view(M, E), G)
            for _ in range(4):
                opts = dict(mode=rng.choice([0, 1]), bg=rng.choice([0, 2]), early=rng.choice([0, 2]), tab=rng.random() < 0.5)
                if seed >= 6:
                    opts.update(head=rng.choice([0, 1]), fused=rng.choice([0, 1]))
                    B.moe_set_option(g.ctx, B.MOE_OPT_HEAD_UNITS, opts["head"])
                    B.moe_set_option(g.ctx, B.MOE_OPT_FUSED_DISPATCH, opts["fused"])
                B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, opts["mode"])
                B.moe_set_option(g.ctx, B.MOE_OPT_BACKGROUND_LANES, opts["bg"])
                B.moe_set_option(g.ctx, B.MOE_OPT_EARLY_SHARED, opts["early"])
                B.moe_set_block_table(g.ctx, table if opts["tab"] else None, -(-E // G))
                out, out2 = g.forward(x, tenant, G), g.forward(x, tenant, G)
                assert B.moe_last_status(g.ctx)[0] == 0, (wl, opts)
                assert torch.equal(out, base) and torch.equal(out2, base), (wl, opts)
        finally:
            g.close()


def _modes_case(name):
    if name == "small-pool":
        wl = W.MoEWorkload("small-pool", T=333, H=256, E=12, I=128, k=3, Is=256, M=3, n_tenants=5, G=5,
                           zipf_bias=True, tenant_layout="uniform")
        return wl, W.make_weights(wl, seed=3, shuffle_slots=True), 3
    if name == "decode":
        wl = W.WORKLOADS["decode"]
        return wl, dict(W.make_weights(W.WORKLOADS["prefill"], seed=0), router_bias=None), 0
    wl = W.scaled(W.WORKLOADS["prefill"], T=1500, n_tenants=6, tenant_layout="uniform")
    return wl, W.make_weights(W.WORKLOADS["prefill"], seed=0), 12


@pytest.mark.parametrize("case", ["small-pool", "decode", "prefill-6-tenants"])
def test_shared_and_private_orchestrator_modes(case):
    # Orchestrator placement: with private orchestrators every tenant's rows of an expert are a request of their own.
    # Invocation counts and the number of row tiles follow the oracle's accounting in both modes; the permutation,
    # the tables and every output bit are the same in both (the row order does not change), and equal the oracle.
    wl, wts, seed = _modes_case(case)
    x, tenant, mot = W.make_tokens(wl, seed=seed)
    T = x.shape[0]
    g = GpuLayer(wl, [wts], T, model_of_tenant=mot)
    try:
        res = {}
        for mode in (B.MOE_DISPATCH_SHARED, B.MOE_DISPATCH_PRIVATE):
            B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, mode)
            o = g.four_calls(x, tenant, wl.G)
            n_tiles, n_stiles, tile_rows = B.moe_last_plan(g.ctx, T)
            f = g.forward(x, tenant, wl.G)
            st = B.moe_last_status(g.ctx)
            assert st[0] == 0 and st[1] == o["n_invocations"] and torch.equal(f, o["out"])
            assert B.moe_last_plan(g.ctx, T)[0] == n_tiles
            acc = oracle.invocations(o["topk_idx"].cpu().numpy(), tenant.numpy(), mot.numpy(), n_models=wl.M, E=wl.E,
                                     G=wl.G, mode=mode, batch_rows=tile_rows)
            assert o["n_invocations"] == acc.n_invocations, (mode, o["n_invocations"], acc.n_invocations)
            assert n_tiles == acc.n_row_batches, (mode, n_tiles, acc.n_row_batches, tile_rows)
            res[mode] = (o, acc)
        o_s, a_s = res[B.MOE_DISPATCH_SHARED]
        o_p, a_p = res[B.MOE_DISPATCH_PRIVATE]
        for key in ("topk_idx", "perm", "inv_perm", "tenant_expert_count", "expert_off", "group_off", "y_perm",
                    "y_shared", "out"):
            if o_s[key] is not None:
                assert torch.equal(o_s[key], o_p[key]), key
        assert a_p.n_invocations > a_s.n_invocations and a_p.n_row_batches > a_s.n_row_batches
        ref = oracle_layer(wl, wts, x, tenant, mot, wl.G, o_p["topk_idx"].cpu().numpy(), o_p["topk_w"].cpu().numpy())
        o_p["n_invocations"] = o_s["n_invocations"]        # (the oracle's dispatch counts the shared placement)
        compare_four_calls(o_p, ref, wl, x)
    finally:
        g.close()


@pytest.mark.parametrize("case", ["small-pool", "decode", "prefill-6-tenants"])
def test_load_aware_block_table(case):
    # Blocks formed from the observed expert loads (greedy, heaviest expert first) instead of ranges of G consecutive
    # experts: the library's host routine equals the oracle's bit for bit; with the table set, the permutation and
    # every output bit are unchanged, the invocation counts and the rows per block follow the oracle's table
    # accounting in both orchestrator modes, and the blocks are more even than the ranges.
    wl, wts, seed = _modes_case(case)
    x, tenant, mot = W.make_tokens(wl, seed=seed)
    T, G, E, M = x.shape[0], max(wl.G, 4), wl.E, wl.M
    Bn = -(-E // G)
    g = GpuLayer(wl, [wts], T, model_of_tenant=mot)
    try:
        base = g.four_calls(x, tenant, G)
        idx = base["topk_idx"].cpu().numpy()
        cnt = base["tenant_expert_count"].cpu().numpy().astype(np.int64)           # [n_tenants, E]
        load = np.zeros((M, E), np.int64)
        for u in range(wl.n_tenants):
            load[int(mot[u])] += cnt[u]
        table = B.moe_form_blocks(torch.from_numpy(load), G)
        ref_table = oracle.form_blocks(load, G=G)
        assert np.array_equal(table.numpy(), ref_table)
        B.moe_set_block_table(g.ctx, table, Bn)
        for mode in (B.MOE_DISPATCH_SHARED, B.MOE_DISPATCH_PRIVATE):
            B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, mode)
            o = g.four_calls(x, tenant, G)
            f = g.forward(x, tenant, G)
            assert o["status"] == 0 and torch.equal(f, base["out"])
            for key in ("topk_idx", "perm", "inv_perm", "tenant_expert_count", "expert_off", "y_perm", "y_shared", "out"):
                if base[key] is not None:
                    assert torch.equal(o[key], base[key]), key
            acc = oracle.invocations_table(idx, tenant.numpy(), mot.numpy(), ref_table, n_blocks=Bn, mode=mode)
            assert o["n_invocations"] == acc.n_invocations
            goff = o["group_off"].cpu().numpy()
            assert np.array_equal(np.diff(goff), acc.block_rows.reshape(-1)) and goff[0] == 0 and goff[-1] == T * wl.k
        rows_table = acc.block_rows.max(axis=1)
        rows_ranges = np.stack([load[:, b * G:(b + 1) * G].sum(axis=1) for b in range(Bn)], axis=1).max(axis=1)
        assert (rows_table <= rows_ranges).all()
        # back to ranges
        B.moe_set_block_table(g.ctx, None)
        B.moe_set_option(g.ctx, B.MOE_OPT_DISPATCH_MODE, B.MOE_DISPATCH_SHARED)
        again = g.four_calls(x, tenant, G)
        assert torch.equal(again["group_off"], base["group_off"]) and again["n_invocations"] == base["n_invocations"]
        assert torch.equal(again["out"], base["out"])
    finally:
        g.close()


def test_on_demand_residency_matches_resident_layer_and_the_lru_oracle():
    # All experts parked in host memory, 6 device slots for 2 x 12 experts: a sequence of small batches (each routes to
    # at most 6 experts) through the paged entry point.  Outputs must equal, bit for bit, a context that keeps every
    # expert resident; hits, loads and evictions per call, and the slot every expert ends up in, must follow the
    # oracle's least-recently-used simulation of the same sequence of active sets.
    wl = W.MoEWorkload("paged", T=3, H=256, E=12, I=128, k=2, Is=128, M=2, n_tenants=3, G=3, tenant_layout="uniform")
    wts = W.make_weights(wl, seed=13)
    mot = W.make_tokens(wl, seed=0)[2]
    full = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    S = 6
    paged = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=wl.T, n_slots=S)
    try:
        dev = paged.device
        shared_only = dict(wts, pool_gate=torch.zeros((S, wl.I, wl.H), dtype=torch.bfloat16),
                           pool_up=torch.zeros((S, wl.I, wl.H), dtype=torch.bfloat16),
                           pool_down=torch.zeros((S, wl.H, wl.I), dtype=torch.bfloat16))
        paged.set_layer_weights(0, shared_only)
        paged.set_tables(model_of_tenant=mot)
        pool = [torch.zeros((S, wl.I, wl.H), dtype=torch.bfloat16, device=dev), torch.zeros((S, wl.I, wl.H), dtype=torch.bfloat16, device=dev),
                torch.zeros((S, wl.H, wl.I), dtype=torch.bfloat16, device=dev)]
        host = [wts["pool_gate"].contiguous().pin_memory(), wts["pool_up"].contiguous().pin_memory(),
                wts["pool_down"].contiguous().pin_memory()]
        B.moe_residency_enable(paged.ctx, 0, host[0], host[1], host[2], pool[0], pool[1], pool[2])
        active_sets, stats = [], []
        seeds = [0, 1, 2, 0, 3, 4, 1, 5, 0, 6]
        for sd in seeds:
            x, tenant, _ = W.make_tokens(wl, seed=sd)
            ref = full.forward(x, tenant, wl.G)
            xd, td = x.to(dev), tenant.to(dev)
            out = torch.zeros_like(xd)
            st = B.moe_layer_forward_paged(paged.ctx, 0, xd, td, wl.T, wl.G, out)
            torch.cuda.synchronize()
            assert B.moe_last_status(paged.ctx)[0] == 0
            assert torch.equal(out, ref), f"batch seed {sd}"
            ws = B.moe_get_workspace(paged.ctx)
            idx = B.wrap_device_pointer(ws["topk_idx"], (wl.T, wl.k), torch.int32, dev).cpu().numpy()
            active_sets.append(sorted({int(mot[tenant[t]]) * wl.E + int(e) for t in range(wl.T) for e in idx[t]}))
            stats.append(st)
        sim = oracle.residency_lru(active_sets, S)
        for st, (h, l, ev, _), need in zip(stats, sim, active_sets):
            assert st == (len(need), h, l, ev), (st, (len(need), h, l, ev))
        assert sum(s[3] for s in stats) > 0 and sum(s[1] for s in stats) > 0       # the sequence did evict and did hit
        # every expert the last batch needed sits in the slot the simulation says, with its own weights
        for e, slot in sim[-1][3].items():
            assert torch.equal(pool[0][slot].cpu(), wts["pool_gate"][e]) and torch.equal(pool[2][slot].cpu(), wts["pool_down"][e])
        # too many active experts for the slots: refused, nothing half done
        wl_big = W.scaled(wl, T=16)
        xb, tb, _ = W.make_tokens(wl_big, seed=7)
        big = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=16, n_slots=4)
        try:
            big.set_layer_weights(0, dict(shared_only, pool_gate=shared_only["pool_gate"][:4], pool_up=shared_only["pool_up"][:4],
                                          pool_down=shared_only["pool_down"][:4]))
            big.set_tables(model_of_tenant=mot)
            pb = [p_[:4].clone() for p_ in pool]
            B.moe_residency_enable(big.ctx, 0, host[0], host[1], host[2], pb[0], pb[1], pb[2])
            with pytest.raises(B.MoeError) as e:
                B.moe_layer_forward_paged(big.ctx, 0, xb.to(dev), tb.to(dev), 16, wl.G, torch.zeros((16, wl.H), dtype=torch.bfloat16, device=dev))
            assert e.value.status == B.MOE_ERR_UNSUPPORTED
        finally:
            big.close()
    finally:
        paged.close()
        full.close()


def test_host_entry_point_matches_device_entry_point():
    wl = W.WORKLOADS["tiny"]
    wts = W.make_weights(wl, seed=0)
    x, tenant, mot = W.make_tokens(wl, seed=0)
    g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    try:
        assert torch.equal(g.forward_host(x, tenant, 1), g.forward(x, tenant, 1).cpu())
    finally:
        g.close()


def test_pipelined_host_calls_match_single_calls():
    # submit / wait with two calls in flight: inputs of a call travel while the previous one computes; every ticket's
    # output must be what the one-call-at-a-time entry point gives for the same batch, whatever the waiting order
    wl = W.MoEWorkload("pipe", T=300, H=256, E=12, I=128, k=3, Is=256, M=2, n_tenants=3, G=4, zipf_bias=True,
                       tenant_layout="uniform")
    wts = W.make_weights(wl, seed=17)
    mot = W.make_tokens(wl, seed=0)[2]
    g = GpuLayer(wl, [wts], wl.T, model_of_tenant=mot)
    try:
        batches = [W.make_tokens(wl, seed=s_)[:2] for s_ in range(7)]
        want = [g.forward_host(x, t, wl.G) for x, t in batches]
        xs = [x.contiguous().pin_memory() for x, _ in batches]
        ts = [t.contiguous().pin_memory() for _, t in batches]
        outs = [torch.zeros_like(x).pin_memory() for x in xs]
        tickets = [B.moe_layer_forward_host_submit(g.ctx, 0, xs[i], ts[i], wl.T, wl.G, outs[i]) for i in range(7)]
        assert tickets == list(range(tickets[0], tickets[0] + 7))
        for i in (6, 0, 3, 5, 1, 2, 4):                  # any order; earlier tickets are complete once a later one is
            B.moe_layer_forward_host_wait(g.ctx, tickets[i])
            assert torch.equal(outs[i], want[i]), i
        assert B.moe_last_status(g.ctx)[0] == 0
        # and the single-call entry point still works afterwards
        assert torch.equal(g.forward_host(*batches[2], wl.G), want[2])
        with pytest.raises(B.MoeError):
            B.moe_layer_forward_host_wait(g.ctx, tickets[-1] + 1)
    finally:
        g.close()


def test_edge_cases_and_errors():
    wl = W.MoEWorkload("edge", T=5, H=256, E=8, I=128, k=2, Is=128, M=1, n_tenants=3)
    wts = W.make_weights(wl, seed=9)
    x, tenant, mot = W.make_tokens(wl, seed=9)
    g = GpuLayer(wl, [wts], 64, model_of_tenant=mot)
    try:
        dev = g.dev
        out = torch.zeros((5, wl.H), dtype=torch.bfloat16, device=dev)
        xd, td = x.to(dev), tenant.to(dev)
        # T = 0 is a no-op
        B.moe_layer_forward(g.ctx, 0, xd, td, 0, 1, out)
        # a single token
        one = g.forward(x[:1].contiguous(), tenant[:1].contiguous(), 1)
        full = g.forward(x, tenant, 1)
        assert torch.equal(one[0], full[0])
        ref = oracle_layer(wl, wts, x, tenant, mot, 1)
        assert_close("edge out", bf16_to_f64(full), ref.out)
        # host-detectable errors launch nothing
        n0 = B.moe_launch_count(g.ctx)
        for G in (0, wl.E + 1):
            with pytest.raises(B.MoeError) as e:
                B.moe_layer_forward(g.ctx, 0, xd, td, 5, G, out)
            assert e.value.status == B.MOE_ERR_G
        with pytest.raises(B.MoeError) as e:
            B.moe_layer_forward(g.ctx, 0, xd, td, 65, 1, out)
        assert e.value.status == B.MOE_ERR_SHAPE
        with pytest.raises(B.MoeError) as e:
            B.moe_layer_forward(g.ctx, 1, xd, td, 5, 1, out)
        assert e.value.status == B.MOE_ERR_SHAPE
        with pytest.raises(B.MoeError) as e:
            B.moe_layer_forward(g.ctx, 0, None, td, 5, 1, out)
        assert e.value.status == B.MOE_ERR_NULL
        assert B.moe_launch_count(g.ctx) == n0
        # activation and output pointers that are not 16-byte aligned are refused on the host: nothing is launched
        # (a kernel given one would fault on its vector loads)
        off_x = torch.zeros(5 * wl.H + 8, dtype=torch.bfloat16, device=dev)[1:1 + 5 * wl.H].view(5, wl.H)
        off_f = torch.zeros(10 * wl.H + 4, dtype=torch.float32, device=dev)[1:1 + 10 * wl.H].view(10, wl.H)
        assert off_x.data_ptr() % 16 == 2 and off_f.data_ptr() % 16 == 4
        o4 = g.four_calls(x, tenant, 1)
        n0 = B.moe_launch_count(g.ctx)
        calls = [
            lambda: B.moe_layer_forward(g.ctx, 0, off_x, td, 5, 1, out),
            lambda: B.moe_layer_forward(g.ctx, 0, xd, td, 5, 1, off_x),
            lambda: B.moe_route(g.ctx, 0, off_x, td, 5, o4["topk_idx"], o4["topk_w"], o4["shared_gate"], o4["tie_flag"]),
            lambda: B.moe_dispatch(g.ctx, off_x, o4["topk_idx"], td, 5, 1, o4["perm"], o4["inv_perm"],
                                   o4["tenant_expert_count"], o4["expert_off"], o4["group_off"], o4["x_perm"]),
            lambda: B.moe_dispatch(g.ctx, xd, o4["topk_idx"], td, 5, 1, o4["perm"], o4["inv_perm"],
                                   o4["tenant_expert_count"], o4["expert_off"], o4["group_off"], off_x),
            lambda: B.moe_experts(g.ctx, 0, xd, o4["x_perm"], o4["perm"], o4["expert_off"], td, 5, 1, off_f, o4["y_shared"]),
            lambda: B.moe_combine(g.ctx, off_f, o4["inv_perm"], o4["topk_w"], o4["y_shared"], o4["shared_gate"], 5, out),
            lambda: B.moe_combine(g.ctx, o4["y_perm"], o4["inv_perm"], o4["topk_w"], o4["y_shared"], o4["shared_gate"], 5,
                                  off_x),
        ]
        for call in calls:
            with pytest.raises(B.MoeError) as e:
                call()
            assert e.value.status == B.MOE_ERR_SHAPE
        assert B.moe_launch_count(g.ctx) == n0
        torch.cuda.synchronize()
        assert B.moe_last_status(g.ctx)[0] == 0
        # an out-of-range tenant id is reported through the status word; that token's output is zero
        bad = tenant.clone(); bad[2] = 7
        outb = g.forward(x, bad, 1)
        st = B.moe_last_status(g.ctx)[0]
        assert st & B.MOE_DEV_BAD_TENANT
        assert torch.count_nonzero(outb[2]) == 0
        keep = [0, 1, 3, 4]
        assert torch.equal(outb[keep], full[keep])
        assert B.moe_last_status(g.ctx)[0] == 0          # cleared by the read
    finally:
        g.close()
    # weights not set -> MOE_ERR_STATE
    ctx = B.moe_create(hidden=256, n_experts=8, inter=128, top_k=2, max_tokens=8)
    try:
        t = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(B.MoeError) as e:
            B.moe_layer_forward(ctx, 0, t, torch.zeros(8, dtype=torch.int32, device="cuda"), 8, 1, t)
        assert e.value.status == B.MOE_ERR_STATE
    finally:
        B.moe_destroy(ctx)
    for kw in (dict(hidden=250), dict(top_k=9), dict(n_experts=0), dict(inter=100)):
        args = dict(hidden=256, n_experts=8, inter=128, top_k=2, max_tokens=8)
        args.update(kw)
        with pytest.raises(B.MoeError):
            B.moe_create(**args)
