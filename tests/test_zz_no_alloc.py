"""The allocation-free dispatch entry point against the regular one.

moe_dispatch_noalloc serves callers that may not allocate device memory (a fixed memory pool, a
latency-critical path, a spent budget) and therefore cannot even create a context.  Its scratch is
a fixed array inside the library that every call shares and that keeps the previous call's
contents, so the check runs two different problems back to back: stale scratch from the first
must not leak into the second.  All outputs are integers, so they must equal moe_dispatch's
bit for bit.  This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import pytest
import torch

from paper_2604_26881_b200 import binding as B

pytestmark = pytest.mark.gpu


def _problem(seed, T, k, E, M, n_tenants, dev):
    g = torch.Generator().manual_seed(seed)
    tenant = torch.randint(0, n_tenants, (T,), generator=g).to(torch.int32)
    idx = torch.stack([torch.randperm(E, generator=g)[:k] for _ in range(T)]).to(torch.int32)
    mot = (torch.arange(n_tenants) % M).to(torch.int32)
    return idx.to(dev), tenant.to(dev), mot


def _outputs(T, k, E, M, n_tenants, G, dev):
    Bn = -(-E // G)
    mk = lambda n: torch.full((n,), -3, dtype=torch.int32, device=dev)
    return dict(perm=mk(T * k), inv_perm=mk(T * k), tenant_expert_count=mk(n_tenants * E), expert_off=mk(M * E + 1),
                group_off=mk(M * Bn + 1))


def _run_both(seed, T, k, E, M, n_tenants, G, dev):
    idx, tenant, mot = _problem(seed, T, k, E, M, n_tenants, dev)
    # reference: the context-based entry point (hidden/inter are irrelevant to the dispatch)
    ctx = B.moe_create(hidden=128, n_experts=E, inter=128, top_k=k, n_models=M, n_tenants=n_tenants, max_tokens=T)
    try:
        B.moe_set_tenant_models(ctx, mot)
        ref = _outputs(T, k, E, M, n_tenants, G, dev)
        B.moe_dispatch(ctx, None, idx, tenant, T, G, ref["perm"], ref["inv_perm"], ref["tenant_expert_count"],
                       ref["expert_off"], ref["group_off"], None)
        torch.cuda.synchronize()
        assert B.moe_last_status(ctx)[0] == 0
    finally:
        B.moe_destroy(ctx)
    got = _outputs(T, k, E, M, n_tenants, G, dev)
    status = torch.full((1,), 99, dtype=torch.int32, device=dev)
    B.moe_dispatch_noalloc(idx, tenant, mot.to(dev), T, k, E, M, n_tenants, G, got["perm"], got["inv_perm"],
                           got["tenant_expert_count"], got["expert_off"], got["group_off"], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for name in ref:
        assert torch.equal(got[name], ref[name]), f"{name} differs from moe_dispatch"
    assert sorted(got["perm"].tolist()) == list(range(T * k))


def test_noalloc_dispatch_matches_dispatch_on_two_calls_in_a_row():
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    # first call: several histogram blocks, several models and tenants, G not dividing E
    _run_both(seed=1, T=1500, k=4, E=60, M=3, n_tenants=7, G=7, dev=dev)
    # second call straight after, smaller and differently shaped: must not see the first call's scratch
    _run_both(seed=2, T=37, k=2, E=8, M=1, n_tenants=2, G=1, dev=dev)
    # and the first shape again with other data
    _run_both(seed=3, T=1500, k=4, E=60, M=3, n_tenants=7, G=60, dev=dev)


def test_noalloc_dispatch_of_an_empty_batch_clears_the_status_word():
    dev = torch.device("cuda:0")
    z = torch.zeros(8, dtype=torch.int32, device=dev)
    status = torch.full((1,), 99, dtype=torch.int32, device=dev)
    B.moe_dispatch_noalloc(z, z, z, 0, 2, 8, 1, 1, 1, z, z, None, z, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0


def test_noalloc_dispatch_rejects_what_does_not_fit():
    dev = torch.device("cuda:0")
    z = torch.zeros(8, dtype=torch.int32, device=dev)
    # 256 experts x 32 tenants = 8192 bins; 2^20 rows -> 4096 histogram blocks: far beyond 2^18 words
    with pytest.raises(B.MoeError) as e:
        B.moe_dispatch_noalloc(z, z, z, 1 << 18, 4, 256, 1, 32, 1, z, z, None, z, None, None)
    assert e.value.status == B.MOE_ERR_UNSUPPORTED
    with pytest.raises(B.MoeError) as e:
        B.moe_dispatch_noalloc(z, z, z, 8, 2, 8, 1, 1, 9, z, z, None, z, None, None)
    assert e.value.status == B.MOE_ERR_G
    with pytest.raises(B.MoeError) as e:
        B.moe_dispatch_noalloc(None, z, z, 8, 2, 8, 1, 1, 1, z, z, None, z, None, None)
    assert e.value.status == B.MOE_ERR_NULL
