"""Pins for the fp64 CPU oracle: each check compares it with something other than
itself -- a library routine (numpy matmul / lexsort, scipy softmax / expit,
torch's bf16 cast), brute force over all expert subsets, a closed form computed
in 50-digit decimal arithmetic, or an invariant the paper states (Sec. 3: block
size does not change semantics; experts are stateless; the orchestrator keeps
no cross-request state)."""
import itertools
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import torch
from scipy.special import expit, softmax

import oracle
from paper_2604_26881_b200 import workloads as W

getcontext().prec = 50


def bf16(a):
    """float array -> (uint16 bit patterns, exact float64 values) after bf16 rounding by torch."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return W.as_u16(t), t.to(torch.float64).numpy()


def rand_bf16(rng, shape, std):
    return bf16(rng.standard_normal(shape) * std)


def small_case(seed=0, T=12, H=16, E=6, I=8, k=2, M=1, n_tenants=1, Is=0, bias=False):
    rng = np.random.default_rng(seed)
    c = {}
    c["x_u"], c["x"] = rand_bf16(rng, (T, H), 1.0)
    c["router_w_u"], c["router_w"] = rand_bf16(rng, (M, E, H), 0.3)
    S = M * E
    c["pg_u"], c["pg"] = rand_bf16(rng, (S, I, H), 0.3)
    c["pu_u"], c["pu"] = rand_bf16(rng, (S, I, H), 0.3)
    c["pd_u"], c["pd"] = rand_bf16(rng, (S, H, I), 0.3)
    c["slot"] = rng.permutation(S).astype(np.int32)
    c["tenant"] = rng.integers(0, n_tenants, T).astype(np.int32)
    c["mot"] = (np.arange(n_tenants) % M).astype(np.int32)
    c["bias"] = rng.standard_normal((M, E)).astype(np.float32) if bias else None
    wts = dict(router_w=c["router_w_u"], router_bias=c["bias"], pool_gate=c["pg_u"], pool_up=c["pu_u"],
               pool_down=c["pd_u"], slot_table=c["slot"])
    if Is:
        c["sg_u"], c["sg"] = rand_bf16(rng, (M, H), 0.3)
        c["wsg_u"], c["wsg"] = rand_bf16(rng, (M, Is, H), 0.3)
        c["wsu_u"], c["wsu"] = rand_bf16(rng, (M, Is, H), 0.3)
        c["wsd_u"], c["wsd"] = rand_bf16(rng, (M, H, Is), 0.3)
        wts.update(shared_gate_w=c["sg_u"], ws_gate=c["wsg_u"], ws_up=c["wsu_u"], ws_down=c["wsd_u"])
    c["wts"] = wts
    c.update(T=T, H=H, E=E, I=I, k=k, M=M, Is=Is)
    return c


def np_silu(a):
    return a * expit(a)          # library sigmoid, not the oracle's formula


def np_ffn(x, wg, wu, wd):
    return (np_silu(x @ wg.T) * (x @ wu.T)) @ wd.T


# ----------------------------------------------------------------------------- gating / top-k

def test_route_probs_match_library_softmax_and_matmul():
    c = small_case(seed=1, M=2, n_tenants=3, bias=True)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], c["bias"], None, k=c["k"])
    for t in range(c["T"]):
        m = c["mot"][c["tenant"][t]]
        z = c["router_w"][m] @ c["x"][t] + c["bias"][m].astype(np.float64)
        np.testing.assert_allclose(r.probs[t], softmax(z), rtol=1e-12, atol=0)
    np.testing.assert_allclose(r.probs.sum(1), 1.0, rtol=1e-12)


@pytest.mark.parametrize("E,k", [(5, 1), (6, 2), (8, 3), (7, 7)])
def test_route_topk_is_best_subset_by_brute_force(E, k):
    c = small_case(seed=2 + E, E=E, k=k, T=20)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, None, k=k)
    for t in range(c["T"]):
        p = softmax(c["router_w"][0] @ c["x"][t])
        best = max(itertools.combinations(range(E), k), key=lambda s: sum(p[list(s)]))
        assert set(r.topk_idx[t]) == set(best)
        # returned in descending probability, weights are the raw probabilities
        assert all(p[r.topk_idx[t, j]] >= p[r.topk_idx[t, j + 1]] for j in range(k - 1))
        np.testing.assert_allclose(r.topk_w[t], p[r.topk_idx[t]], rtol=1e-12)
        assert r.topk_w[t].sum() <= 1.0 + 1e-12
        if k < E:
            assert r.topk_w[t].sum() < 1.0       # no renormalisation


def test_route_equal_logits_closed_form_and_tie_break():
    E, k, H, T = 8, 3, 4, 5
    x_u, _ = bf16(np.ones((T, H)))
    w_u, _ = bf16(np.zeros((1, E, H)))
    r = oracle.route(x_u, np.zeros(T, np.int32), np.zeros(1, np.int32), w_u, None, None, k=k)
    assert np.all(r.probs == 1.0 / E)                       # exactly
    assert np.all(r.topk_idx == np.arange(k, dtype=np.int32))   # ties -> lower id first
    assert np.all(r.tie_flag == 1)


def test_route_dominant_logit_and_bias_only_ordering():
    E, k, H = 6, 2, 4
    x_u, _ = bf16(np.ones((1, H)))
    w = np.zeros((1, E, H)); w[0, 4, :] = 12.5       # z_4 = 50
    w_u, _ = bf16(w)
    r = oracle.route(x_u, np.zeros(1, np.int32), np.zeros(1, np.int32), w_u, None, None, k=k)
    assert r.topk_idx[0, 0] == 4 and abs(r.topk_w[0, 0] - 1.0) < 1e-20 + 5 * math.exp(-50) * 1.01
    # with zero router weights the bias alone decides: p = softmax(b)
    b = np.array([[0.5, -1.0, 2.0, 0.25, 1.5, -3.0]], np.float32)
    w0_u, _ = bf16(np.zeros((1, E, H)))
    r = oracle.route(x_u, np.zeros(1, np.int32), np.zeros(1, np.int32), w0_u, b, None, k=3)
    assert list(r.topk_idx[0]) == [2, 4, 0]
    den = sum(Decimal(float(v)).exp() for v in b[0])
    for j, e in enumerate([2, 4, 0]):
        assert abs(Decimal(r.topk_w[0, j]) - Decimal(float(b[0, e])).exp() / den) < Decimal(10) ** -15


def test_route_uses_the_router_of_the_tenants_model():
    c = small_case(seed=5, M=2, n_tenants=4, T=16)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, None, k=2)
    for t in range(c["T"]):
        m = c["tenant"][t] % 2
        np.testing.assert_allclose(r.probs[t], softmax(c["router_w"][m] @ c["x"][t]), rtol=1e-12)
    with pytest.raises(ValueError):
        bad = c["tenant"].copy(); bad[3] = 4
        oracle.route(c["x_u"], bad, c["mot"], c["router_w_u"], None, None, k=2)


def test_route_tie_flag_thresholds():
    E, k, H = 6, 2, 2
    x_u, _ = bf16(np.ones((1, H)))
    w0_u, _ = bf16(np.zeros((1, E, H)))

    def flag(b):
        r = oracle.route(x_u, np.zeros(1, np.int32), np.zeros(1, np.int32), w0_u,
                         np.asarray([b], np.float32), None, k=k)
        return int(r.tie_flag[0])
    # relative gap of p equals 1 - exp(-dz); float32 biases chosen around the 1e-5 threshold
    assert flag([3.0, 2.0, 1.0, 0.0, -1.0, -2.0]) == 0
    assert flag([3.0, 3.0 - 2e-6, 1.0, 0.0, -1.0, -2.0]) == 1          # rank 1 vs 2
    assert flag([3.0, 2.0, 2.0 - 2e-6, 0.0, -1.0, -2.0]) == 1          # rank k vs k+1
    assert flag([3.0, 2.0, 1.0, 1.0 - 2e-6, -1.0, -2.0]) == 0          # beyond rank k+1: irrelevant
    assert flag([3.0, 3.0 - 1e-3, 1.0, 0.0, -1.0, -2.0]) == 0          # gap 1e-3 is resolvable


def test_shared_gate_closed_form_and_library():
    c = small_case(seed=6, Is=8, M=2, n_tenants=2)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, c["sg_u"], k=2)
    ref = np.array([expit(c["sg"][c["mot"][c["tenant"][t]]] @ c["x"][t]) for t in range(c["T"])])
    np.testing.assert_allclose(r.shared_gate, ref, rtol=1e-13)
    z_u, _ = bf16(np.zeros((2, c["H"])))
    r0 = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, z_u, k=2)
    assert np.all(r0.shared_gate == 0.5)


# ----------------------------------------------------------------------------- dispatch

def _lexsort_dispatch(idx, tenant, mot):
    T, k = idx.shape
    rows = np.arange(T * k)
    t = rows // k
    e = idx.reshape(-1)
    u = tenant[t]
    m = mot[u]
    order = np.lexsort((t, u, e, m))      # last key is the primary one
    return rows[order].astype(np.int32)


@pytest.mark.parametrize("seed,M,n_tenants,G", [(0, 1, 1, 1), (1, 1, 4, 2), (2, 2, 5, 3), (3, 3, 3, 6), (4, 2, 7, 4)])
def test_dispatch_matches_lexsort_and_invariants(seed, M, n_tenants, G):
    rng = np.random.default_rng(seed)
    T, E, k = 37, 6, 3
    tenant = rng.integers(0, n_tenants, T).astype(np.int32)
    mot = (np.arange(n_tenants) % M).astype(np.int32)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    d = oracle.dispatch(idx, tenant, mot, n_models=M, E=E, G=G)
    R = T * k
    assert np.array_equal(d.perm, _lexsort_dispatch(idx, tenant, mot))
    assert sorted(d.perm.tolist()) == list(range(R))                 # bijection
    assert np.array_equal(d.inv_perm[d.perm], np.arange(R))          # inverse
    assert d.tenant_expert_count.sum() == R
    for u in range(n_tenants):
        for e in range(E):
            assert d.tenant_expert_count[u, e] == int(np.sum((idx == e).any(1) & (tenant == u)))
    assert np.all(np.bincount(d.perm // k, minlength=T) == k)         # each token k times
    # expert_off is the exclusive scan of per-(model, expert) counts
    cnt_me = np.zeros(M * E + 1, np.int64)
    for u in range(n_tenants):
        cnt_me[mot[u] * E:(mot[u] + 1) * E] += d.tenant_expert_count[u]
    assert np.array_equal(d.expert_off, np.concatenate([[0], np.cumsum(cnt_me[:-1])]))
    B = -(-E // G)
    for m in range(M):
        for b in range(B):
            assert d.group_off[m * B + b] == d.expert_off[m * E + min(b * G, E)]
    assert d.group_off[-1] == R
    nonempty = {(mot[tenant[r // k]], idx.reshape(-1)[r] // G) for r in range(R)}
    assert d.n_invocations == len(nonempty)
    # every row of a segment belongs to that segment's expert and model
    for m in range(M):
        for e in range(E):
            for pos in range(d.expert_off[m * E + e], d.expert_off[m * E + e + 1]):
                row = d.perm[pos]
                assert idx.reshape(-1)[row] == e and mot[tenant[row // k]] == m


def test_dispatch_perm_is_independent_of_G_and_group_tables_nest():
    rng = np.random.default_rng(9)
    T, E, k = 50, 12, 4
    tenant = rng.integers(0, 3, T).astype(np.int32)
    mot = np.zeros(3, np.int32)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    ref = oracle.dispatch(idx, tenant, mot, n_models=1, E=E, G=1)
    assert np.array_equal(ref.group_off, ref.expert_off)              # G = 1: blocks are experts
    for G in (2, 3, 4, 5, 6, 12):
        d = oracle.dispatch(idx, tenant, mot, n_models=1, E=E, G=G)
        assert np.array_equal(d.perm, ref.perm) and np.array_equal(d.inv_perm, ref.inv_perm)
        assert np.array_equal(d.expert_off, ref.expert_off)
    dE = oracle.dispatch(idx, tenant, mot, n_models=1, E=E, G=E)
    assert list(dE.group_off) == [0, T * k] and dE.n_invocations == 1
    with pytest.raises(ValueError):
        oracle.dispatch(idx, tenant, mot, n_models=1, E=E, G=0)
    with pytest.raises(ValueError):
        oracle.dispatch(idx, tenant, mot, n_models=1, E=E, G=E + 1)


def test_dispatch_invocation_count_with_sparse_blocks():
    # experts 1 and 6 of 12 are hit: with G = 4 that is blocks 0 and 1 (whose first experts are empty)
    idx = np.array([[1, 6], [6, 1], [1, 6]], np.int32)
    tenant = np.zeros(3, np.int32); mot = np.zeros(1, np.int32)
    assert oracle.dispatch(idx, tenant, mot, n_models=1, E=12, G=4).n_invocations == 2
    assert oracle.dispatch(idx, tenant, mot, n_models=1, E=12, G=1).n_invocations == 2
    assert oracle.dispatch(idx, tenant, mot, n_models=1, E=12, G=12).n_invocations == 1
    d = oracle.dispatch(idx, tenant, mot, n_models=1, E=12, G=5)          # G need not divide E: last block short
    assert list(d.group_off) == [0, 3, 6, 6] and d.n_invocations == 2


# ----------------------------------------------------------------------------- expert FFN

def test_experts_match_numpy_matmul_restatement():
    c = small_case(seed=11, T=9, H=24, I=10, E=5, k=2, M=2, n_tenants=3)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, None, k=2)
    d = oracle.dispatch(r.topk_idx, c["tenant"], c["mot"], n_models=2, E=5, G=1)
    y = oracle.experts(c["x_u"], c["tenant"], r.topk_idx, d.perm, c["mot"], c["pg_u"], c["pu_u"], c["pd_u"],
                       c["slot"], n_models=2)
    for pos, row in enumerate(d.perm):
        t, j = divmod(int(row), 2)
        s = c["slot"][c["mot"][c["tenant"][t]] * 5 + r.topk_idx[t, j]]
        ref = np_ffn(c["x"][t], c["pg"][s], c["pu"][s], c["pd"][s])
        np.testing.assert_allclose(y[pos], ref, rtol=1e-11, atol=1e-13)


def test_swiglu_scalar_closed_form_in_decimal():
    # H = I = 1: y = wd * silu(wg*x) * (wu*x), with silu(a) = a / (1 + e^-a) evaluated in 50 digits
    for x, wg, wu, wd in [(1.0, 0.5, 2.0, -1.5), (-2.0, 1.25, 0.75, 3.0), (0.375, -4.0, -0.5, 0.125)]:
        x_u, _ = bf16([[x]]); g_u, _ = bf16([[[wg]]]); u_u, _ = bf16([[[wu]]]); d_u, _ = bf16([[[wd]]])
        y = oracle.experts(x_u, np.zeros(1, np.int32), np.zeros((1, 1), np.int32), np.zeros(1, np.int32),
                           np.zeros(1, np.int32), g_u, u_u, d_u, np.zeros(1, np.int32), n_models=1)
        a = Decimal(wg) * Decimal(x)
        ref = Decimal(wd) * (a / (1 + (-a).exp())) * (Decimal(wu) * Decimal(x))
        assert abs(Decimal(float(y[0, 0])) - ref) < abs(ref) * Decimal(10) ** -14


def test_experts_zero_cases():
    c = small_case(seed=12)
    r = oracle.route(c["x_u"], c["tenant"], c["mot"], c["router_w_u"], None, None, k=2)
    d = oracle.dispatch(r.topk_idx, c["tenant"], c["mot"], n_models=1, E=c["E"], G=1)
    zero_d = np.zeros_like(c["pd_u"])
    y = oracle.experts(c["x_u"], c["tenant"], r.topk_idx, d.perm, c["mot"], c["pg_u"], c["pu_u"], zero_d,
                       c["slot"], n_models=1)
    assert np.all(y == 0)
    y = oracle.experts(np.zeros_like(c["x_u"]), c["tenant"], r.topk_idx, d.perm, c["mot"], c["pg_u"], c["pu_u"],
                       c["pd_u"], c["slot"], n_models=1)
    assert np.all(y == 0)


def test_shared_expert_equals_sum_of_four_narrow_experts():
    # a SwiGLU of width 4*I is the sum of 4 SwiGLUs over consecutive slices of the intermediate axis
    c = small_case(seed=13, Is=16, H=12, T=7)
    ys = oracle.shared_expert(c["x_u"], c["tenant"], c["mot"], c["wsg_u"], c["wsu_u"], c["wsd_u"])
    acc = np.zeros_like(ys)
    for q in range(4):
        sl = slice(4 * q, 4 * q + 4)
        acc += oracle.shared_expert(c["x_u"], c["tenant"], c["mot"],
                                    np.ascontiguousarray(c["wsg_u"][:, sl]), np.ascontiguousarray(c["wsu_u"][:, sl]),
                                    np.ascontiguousarray(c["wsd_u"][:, :, sl]))
    np.testing.assert_allclose(ys, acc, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(ys, np_ffn(c["x"], c["wsg"][0], c["wsu"][0], c["wsd"][0]), rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------- whole layer

def _layer(c, G=1, tenant=None, x_u=None, **kw):
    return oracle.layer_forward(c["x_u"] if x_u is None else x_u, c["tenant"] if tenant is None else tenant,
                                c["mot"], c["wts"], k=c["k"], G=G, **kw)


def test_layer_single_expert_is_plain_ffn():
    c = small_case(seed=20, E=1, k=1)
    res = _layer(c)
    assert np.all(res.routing.topk_w == 1.0)
    np.testing.assert_allclose(res.out, np_ffn(c["x"], c["pg"][0], c["pu"][0], c["pd"][0]), rtol=1e-11, atol=1e-13)


def test_layer_k_equals_E_is_dense_soft_mixture():
    c = small_case(seed=21, E=4, k=4)
    res = _layer(c)
    p = softmax(c["x"] @ c["router_w"][0].T, axis=1)
    ref = sum(p[:, [e]] * np_ffn(c["x"], c["pg"][c["slot"][e]], c["pu"][c["slot"][e]], c["pd"][c["slot"][e]])
              for e in range(4))
    np.testing.assert_allclose(res.out, ref, rtol=1e-11, atol=1e-13)


def test_layer_equals_brute_force_best_subset_with_shared_expert():
    c = small_case(seed=22, E=6, k=3, Is=8, M=2, n_tenants=3, bias=True)
    res = _layer(c)
    for t in range(c["T"]):
        m = c["mot"][c["tenant"][t]]
        p = softmax(c["router_w"][m] @ c["x"][t] + c["bias"][m].astype(np.float64))
        best = max(itertools.combinations(range(6), 3), key=lambda s: sum(p[list(s)]))
        ref = sum(p[e] * np_ffn(c["x"][t], *(c[n][c["slot"][m * 6 + e]] for n in ("pg", "pu", "pd"))) for e in best)
        ref = ref + expit(c["sg"][m] @ c["x"][t]) * np_ffn(c["x"][t], c["wsg"][m], c["wsu"][m], c["wsd"][m])
        np.testing.assert_allclose(res.out[t], ref, rtol=1e-10, atol=1e-12)


def test_layer_permuting_tokens_permutes_outputs():
    c = small_case(seed=23, n_tenants=3, Is=8)
    res = _layer(c)
    pi = np.random.default_rng(0).permutation(c["T"])
    res2 = _layer(c, tenant=c["tenant"][pi], x_u=c["x_u"][pi])
    assert np.array_equal(res2.out, res.out[pi])          # bit-identical: tokens are independent


def test_layer_output_identical_for_every_G():
    c = small_case(seed=24, E=6, k=2, M=2, n_tenants=4, Is=8)
    ref = _layer(c, G=1)
    for G in (2, 3, 4, 6):
        r = _layer(c, G=G)
        assert np.array_equal(r.out, ref.out) and np.array_equal(r.dispatch.perm, ref.dispatch.perm)
        assert np.array_equal(r.routing.topk_idx, ref.routing.topk_idx)


def test_layer_split_by_tenant_equals_mixed_batch():
    c = small_case(seed=25, T=24, M=2, n_tenants=4, Is=8)
    mixed = _layer(c)
    for u in range(4):
        sel = np.nonzero(c["tenant"] == u)[0]
        if len(sel) == 0:
            continue
        alone = _layer(c, tenant=c["tenant"][sel], x_u=c["x_u"][sel])
        assert np.array_equal(alone.out, mixed.out[sel])


def test_layer_topk_override_only_touches_masked_tokens():
    c = small_case(seed=26, E=6, k=2)
    base = _layer(c)
    idx_o = base.routing.topk_idx.copy()
    mask = np.zeros(c["T"], bool); mask[3] = True
    idx_o[3] = idx_o[3][::-1]                         # same set, swapped order
    res = _layer(c, topk_override=(idx_o, mask))
    np.testing.assert_allclose(res.out, base.out, rtol=1e-13, atol=1e-15)
    idx_o[3] = [e for e in range(6) if e not in base.routing.topk_idx[3]][:2]
    res = _layer(c, topk_override=(idx_o, mask))
    assert np.array_equal(np.delete(res.out, 3, 0), np.delete(base.out, 3, 0))
    assert not np.allclose(res.out[3], base.out[3])


# ----------------------------------------------------------------------------- stacked blocks

def test_round_bf16_matches_torch_cast_and_ties_to_even():
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    ref = W.as_u16(torch.from_numpy(v).to(torch.bfloat16))         # float32 -> bf16 is a single rounding
    assert np.array_equal(oracle.round_bf16(v.astype(np.float64)), ref)
    # exact halfway points between neighbouring bf16 values: ties go to the even mantissa
    assert oracle.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80          # 1.0 (even) not 1.0078125
    assert oracle.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82      # up to even
    # a double just above the halfway point must round up even though float32 would tie
    assert oracle.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    assert oracle.round_bf16(np.array([-(1.0 + 2.0 ** -8 + 2.0 ** -40)]))[0] == 0xBF81
    assert oracle.round_bf16(np.array([0.0]))[0] == 0


def test_rmsnorm_constant_vector_closed_form():
    H = 64
    for cval in (2.0, -0.5):
        x_u, _ = bf16(np.full((3, H), cval))
        g_u, g = bf16(1.0 + 0.125 * np.arange(H) / H)
        xn = oracle.rmsnorm(x_u, g_u, 1e-6)
        ref = np.sign(cval) * g / math.sqrt(1.0 + 1e-6 / cval ** 2)
        np.testing.assert_allclose(xn, np.broadcast_to(ref, (3, H)), rtol=1e-14)


def test_rmsnorm_matches_numpy_and_zero_weights_make_block_identity():
    c = small_case(seed=30, Is=8)
    g_u, g = bf16(1.0 + 0.02 * np.random.default_rng(1).standard_normal(c["H"]))
    xn = oracle.rmsnorm(c["x_u"], g_u, 1e-6)
    ref = c["x"] / np.sqrt((c["x"] ** 2).mean(1, keepdims=True) + 1e-6) * g
    np.testing.assert_allclose(xn, ref, rtol=1e-13)
    wts = dict(c["wts"]); wts["rms_w"] = g_u
    wts["pool_down"] = np.zeros_like(c["pd_u"]); wts["ws_down"] = np.zeros_like(c["wsd_u"])
    x_next, xn_u, _ = oracle.block_forward(c["x_u"], c["tenant"], c["mot"], wts, k=2, G=1, eps=1e-6)
    assert np.array_equal(x_next, c["x_u"])
    assert np.array_equal(xn_u, oracle.round_bf16(ref)) or np.max(np.abs(
        xn_u.astype(np.int32) - oracle.round_bf16(ref).astype(np.int32))) <= 1


def _nearest_bf16_by_table(v):
    """Round-to-nearest-even onto bf16 by searching the sorted table of all finite bf16 values."""
    bits = np.arange(1 << 16, dtype=np.uint32)
    with np.errstate(invalid="ignore"):
        vals = (bits << 16).view(np.float32).astype(np.float64)
    ok = np.isfinite(vals) & ~((bits == 0x8000))            # one zero
    bits, vals = bits[ok], vals[ok]
    order = np.argsort(vals, kind="stable")
    bits, vals = bits[order], vals[order]
    hi = np.clip(np.searchsorted(vals, v), 1, len(vals) - 1)
    lo = hi - 1
    dl, dh = np.abs(v - vals[lo]), np.abs(vals[hi] - v)
    pick_hi = (dh < dl) | ((dh == dl) & ((bits[hi] & 1) == 0))
    return np.where(pick_hi, bits[hi], bits[lo]).astype(np.uint16)


def test_block_forward_residual_add_with_nonzero_layer_output():
    # x_next = bf16(x + layer(xn)) with a layer output that is far from zero.  The sum is restated with numpy on the
    # exact bf16 values of x and rounded by a table search over all bf16 values (no shared rounding code), so a wrong
    # sign, a dropped summand or a scale on either term fails.
    c = small_case(seed=33, Is=8)
    g_u, _ = bf16(1.0 + 0.02 * np.random.default_rng(2).standard_normal(c["H"]))
    wts = dict(c["wts"]); wts["rms_w"] = g_u
    x_next, xn_u, res = oracle.block_forward(c["x_u"], c["tenant"], c["mot"], wts, k=2, G=1, eps=1e-6)
    assert np.abs(res.out).max() > 1e-2                       # the layer really contributes
    # the layer inside the block ran on the rounded normalised input
    direct = _layer(dict(c, wts=wts), x_u=xn_u)
    assert np.array_equal(direct.out, res.out)
    total = c["x"] + res.out                                   # fp64, exact inputs
    assert np.array_equal(x_next, _nearest_bf16_by_table(total))
    # the classic mistakes give other bits
    for wrong in (c["x"] - res.out, c["x"] + 2 * res.out, res.out, c["x"]):
        assert not np.array_equal(_nearest_bf16_by_table(wrong), x_next)


# ----------------------------------------------------------------------------- orchestrator placement (Sec. 4.2, Sec. 5)

def _brute_invocations(idx, tenant, mot, E, G, mode, batch_rows):
    """Python sets over (tenant, model, block, expert) of every routed row."""
    rows = [(int(tenant[t]), int(mot[tenant[t]]), int(e) // G, int(e)) for t in range(idx.shape[0]) for e in idx[t]]
    if mode == oracle.SHARED:
        inv = {(m, b) for (_, m, b, _) in rows}
        segs = {}
        for (_, m, _, e) in rows:
            segs[(m, e)] = segs.get((m, e), 0) + 1
    else:
        inv = {(u, b) for (u, _, b, _) in rows}
        segs = {}
        for (u, _, _, e) in rows:
            segs[(u, e)] = segs.get((u, e), 0) + 1
    per_tenant = [len({b for (u2, _, b, _) in rows if u2 == u}) for u in range(len(mot))]
    fan = [len({int(e) // G for e in idx[t]}) for t in range(idx.shape[0])]
    batches = sum(-(-c // batch_rows) for c in segs.values())
    return len(inv), per_tenant, fan, batches


def test_invocations_match_brute_force_for_both_orchestrator_placements():
    rng = np.random.default_rng(40)
    for trial in range(60):
        E = int(rng.integers(2, 13)); k = int(rng.integers(1, min(E, 4) + 1)); M = int(rng.integers(1, 4))
        nt = int(rng.integers(M, M + 4)); T = int(rng.integers(1, 40)); G = int(rng.integers(1, E + 1))
        br = int(rng.integers(1, 6))
        idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
        tenant = rng.integers(0, nt, T).astype(np.int32)
        mot = (np.arange(nt) % M).astype(np.int32)
        for mode in (oracle.SHARED, oracle.PRIVATE):
            r = oracle.invocations(idx, tenant, mot, n_models=M, E=E, G=G, mode=mode, batch_rows=br)
            n, per_tenant, fan, batches = _brute_invocations(idx, tenant, mot, E, G, mode, br)
            assert r.n_invocations == n and r.n_row_batches == batches
            assert r.tenant_invocations.tolist() == per_tenant and r.token_fanout.tolist() == fan
        sh = oracle.invocations(idx, tenant, mot, n_models=M, E=E, G=G, mode=oracle.SHARED, batch_rows=br)
        pr = oracle.invocations(idx, tenant, mot, n_models=M, E=E, G=G, mode=oracle.PRIVATE, batch_rows=br)
        # the shared count is what the dispatch reports; private orchestrators can only add invocations, never more
        # than one per tenant and shared invocation; and they are the sum of what each tenant issues
        d = oracle.dispatch(idx, tenant, mot, n_models=M, E=E, G=G)
        assert sh.n_invocations == d.n_invocations
        assert sh.n_invocations <= pr.n_invocations <= sh.n_invocations * nt
        assert pr.n_invocations == int(pr.tenant_invocations.sum())
        assert pr.n_row_batches >= sh.n_row_batches
        # a token takes part in between 1 and min(k, blocks) invocations
        assert fan and min(pr.token_fanout) >= 1 and max(pr.token_fanout) <= min(k, -(-E // G))


def test_private_placement_with_one_tenant_equals_shared_placement():
    rng = np.random.default_rng(41)
    E, k, T = 10, 3, 50
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    tenant = np.zeros(T, np.int32); mot = np.zeros(1, np.int32)
    for G in (1, 3, 10):
        a = oracle.invocations(idx, tenant, mot, n_models=1, E=E, G=G, mode=oracle.SHARED, batch_rows=4)
        b = oracle.invocations(idx, tenant, mot, n_models=1, E=E, G=G, mode=oracle.PRIVATE, batch_rows=4)
        assert a.n_invocations == b.n_invocations and a.n_row_batches == b.n_row_batches
        assert np.array_equal(a.token_fanout, b.token_fanout)
        assert np.array_equal(a.tenant_invocations, b.tenant_invocations)
    # one block holding every expert: one shared invocation per model, one private invocation per tenant with tokens
    tenant = rng.integers(0, 5, T).astype(np.int32); mot = (np.arange(5) % 2).astype(np.int32)
    a = oracle.invocations(idx, tenant, mot, n_models=2, E=E, G=E, mode=oracle.SHARED)
    b = oracle.invocations(idx, tenant, mot, n_models=2, E=E, G=E, mode=oracle.PRIVATE)
    assert a.n_invocations == len(set(mot[tenant])) and b.n_invocations == len(set(tenant.tolist()))
    assert (a.token_fanout == 1).all()
    # G = 1: a token reaches k blocks
    c = oracle.invocations(idx, tenant, mot, n_models=2, E=E, G=1, mode=oracle.PRIVATE)
    assert (c.token_fanout == k).all()


# ----------------------------------------------------------------------------- load-aware block formation (Sec. 5)

def _best_makespan(load, G):
    """Smallest possible largest block load over ALL assignments with at most G experts per block (tiny E only)."""
    import itertools
    E = len(load); B = -(-E // G)
    best = None
    for assign in itertools.product(range(B), repeat=E):
        sizes = [assign.count(b) for b in range(B)]
        if max(sizes) > G:
            continue
        ms = max(sum(load[e] for e in range(E) if assign[e] == b) for b in range(B))
        best = ms if best is None or ms < best else best
    return best


def test_form_blocks_hand_worked_example_and_structure():
    # loads 10 9 8 7 1 1, blocks of 2: 10 -> b0, 9 -> b1, 8 -> b2, 7 -> lightest with room = b2 (8), 1 -> b1 (9),
    # 1 -> b0 (10): worked by hand from the rule
    blk = oracle.form_blocks(np.array([[10, 9, 8, 7, 1, 1]]), G=2)
    assert blk.tolist() == [[0, 1, 2, 2, 1, 0]]
    # equal loads: ties go to the lower expert id and the lower block id, so the experts are dealt round robin
    assert oracle.form_blocks(np.full((1, 6), 5), G=2).tolist() == [[0, 1, 2, 0, 1, 2]]
    # G = 1: every expert its own block; G = E: one block
    l = np.array([[3, 9, 1, 4]])
    assert sorted(oracle.form_blocks(l, G=1)[0].tolist()) == [0, 1, 2, 3]
    assert oracle.form_blocks(l, G=4).tolist() == [[0, 0, 0, 0]]
    # models are independent
    two = oracle.form_blocks(np.array([[10, 9, 8, 7, 1, 1], [1, 1, 7, 8, 9, 10]]), G=2)
    # (second model: 10 -> b0, 9 -> b1, 8 -> b2, 7 -> b2, then expert 0 before expert 1: 1 -> b1 (9), 1 -> b0 (10))
    assert two[0].tolist() == [0, 1, 2, 2, 1, 0] and two[1].tolist() == [1, 0, 2, 2, 1, 0]


def test_form_blocks_is_a_partition_with_capacity_and_close_to_the_best_assignment():
    rng = np.random.default_rng(50)
    for trial in range(150):
        E = int(rng.integers(2, 8)); G = int(rng.integers(1, E + 1)); B = -(-E // G)
        load = rng.integers(0, 30, E)
        if trial % 2:
            load = (30 / np.arange(1, E + 1) ** 1.1).astype(np.int64)[rng.permutation(E)]      # Zipf-like skew
        blk = oracle.form_blocks(load[None], G=G)[0]
        assert blk.min() >= 0 and blk.max() < B
        assert np.bincount(blk, minlength=B).max() <= G
        ms = max(int(load[blk == b].sum()) for b in range(B))
        best = _best_makespan(load.tolist(), G)
        assert best <= ms <= best * 4 / 3 + 1e-9, (load, G, blk, ms, best)
        # never worse than the blocks of G consecutive experts on their best day: the heaviest expert bounds both
        assert ms >= load.max()
    # on a Zipf-skewed load the greedy blocks are more even than blocks of consecutive experts
    load = (4096 * 4 / np.arange(1, 61) ** 1.1)
    load = (load / load.sum() * 16384).astype(np.int64)[np.random.default_rng(1).permutation(60)]
    blk = oracle.form_blocks(load[None], G=4)[0]
    greedy = max(int(load[blk == b].sum()) for b in range(15))
    ranges = max(int(load[b * 4:(b + 1) * 4].sum()) for b in range(15))
    assert greedy <= ranges and greedy == max(int(load.max()), greedy)


def test_invocations_table_equals_range_accounting_for_range_tables_and_brute_force_otherwise():
    rng = np.random.default_rng(51)
    for trial in range(40):
        E = int(rng.integers(2, 13)); k = int(rng.integers(1, min(E, 4) + 1)); M = int(rng.integers(1, 4))
        nt = int(rng.integers(M, M + 4)); T = int(rng.integers(1, 40)); G = int(rng.integers(1, E + 1)); B = -(-E // G)
        idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
        tenant = rng.integers(0, nt, T).astype(np.int32)
        mot = (np.arange(nt) % M).astype(np.int32)
        ranges = np.tile((np.arange(E) // G).astype(np.int32), (M, 1))
        table = np.stack([rng.permutation(np.arange(E) % B) for _ in range(M)]).astype(np.int32)
        for mode in (oracle.SHARED, oracle.PRIVATE):
            a = oracle.invocations(idx, tenant, mot, n_models=M, E=E, G=G, mode=mode)
            b = oracle.invocations_table(idx, tenant, mot, ranges, n_blocks=B, mode=mode)
            assert a.n_invocations == b.n_invocations and np.array_equal(a.token_fanout, b.token_fanout)
            assert np.array_equal(a.tenant_invocations, b.tenant_invocations)
            c = oracle.invocations_table(idx, tenant, mot, table, n_blocks=B, mode=mode)
            rows = [(int(tenant[t]), int(mot[tenant[t]]), int(table[mot[tenant[t]], e])) for t in range(T) for e in idx[t]]
            want = len({(m, bb) for (_, m, bb) in rows}) if mode == oracle.SHARED else len({(u, bb) for (u, _, bb) in rows})
            assert c.n_invocations == want
            assert c.block_rows.sum() == T * k
            for m in range(M):
                for bb in range(B):
                    assert c.block_rows[m, bb] == sum(1 for (_, m2, b2) in rows if m2 == m and b2 == bb)
            assert c.token_fanout.tolist() == [len({int(table[mot[tenant[t]], e]) for e in idx[t]}) for t in range(T)]


# ----------------------------------------------------------------------------- on-demand residency (abstract, Sec. 3)

def _min_loads(seq, n_slots):
    """Fewest loads any eviction policy needs (exhaustive search over the victims; tiny sequences only)."""
    import functools

    @functools.lru_cache(maxsize=None)
    def go(step, resident):
        if step == len(seq):
            return 0
        need = frozenset(seq[step])
        res = set(resident)
        missing = sorted(need - res)
        if not missing:
            return go(step + 1, resident)
        best = None

        def place(i, cur):
            nonlocal best
            if i == len(missing):
                v = len(missing) + go(step + 1, frozenset(cur))
                best = v if best is None or v < best else best
                return
            if len(cur) < n_slots:
                place(i + 1, cur | {missing[i]})
            else:
                for victim in sorted(cur - need):
                    place(i + 1, (cur - {victim}) | {missing[i]})
        place(0, set(res))
        return best
    return go(0, frozenset())


def test_residency_lru_hand_example_and_bounds():
    # two slots; batches {1} {2} {1} {3} {2}: loads 1, 2; hit 1; 3 evicts 2 (needed longest ago); 2 evicts 1
    r = oracle.residency_lru([[1], [2], [1], [3], [2]], 2)
    assert [(h, l, e) for h, l, e, _ in r] == [(0, 1, 0), (0, 1, 0), (1, 0, 0), (0, 1, 1), (0, 1, 1)]
    assert r[3][3] == {1: 0, 3: 1} and r[4][3] == {2: 0, 3: 1}
    # enough slots for everything: every expert is loaded exactly once, nothing is evicted, a repeated batch only hits
    rng = np.random.default_rng(60)
    seq = [sorted(rng.choice(12, 4, replace=False).tolist()) for _ in range(10)]
    seq.append(seq[-1])
    r = oracle.residency_lru(seq, 12)
    assert sum(l for _, l, _, _ in r) == len({e for b in seq for e in b}) and sum(e for _, _, e, _ in r) == 0
    assert r[-1][:3] == (4, 0, 0)
    # any capacity: hits + loads = batch size, the batch is resident afterwards, evictions only when full, and no
    # policy can do with fewer loads than the exhaustive optimum while LRU stays within the classic factor of it
    for trial in range(40):
        S = int(rng.integers(2, 5)); n = int(rng.integers(1, S + 1))
        seq = [sorted(rng.choice(6, n, replace=False).tolist()) for _ in range(7)]
        r = oracle.residency_lru(seq, S)
        resident = set()
        for (h, l, ev, slot_of), need in zip(r, seq):
            assert h == len(set(need) & resident) and h + l == len(need)
            assert set(need) <= set(slot_of) and len(set(slot_of.values())) == len(slot_of) <= S
            assert ev == max(0, len(resident) + l - S)
            resident = set(slot_of)
        total = sum(l for _, l, _, _ in r)
        best = _min_loads(tuple(tuple(b) for b in seq), S)
        assert best <= total <= best * S            # LRU is S-competitive
    with pytest.raises(ValueError):
        oracle.residency_lru([[1, 2, 3]], 2)
