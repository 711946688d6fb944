"""The expert-parallel exchange protocol on a GPU: one rank over NCCL, the library's own expert call as the expert step.

With one GPU the two all-to-alls of `expert_parallel.ExpertParallel` send every row to the rank it came from, so
nothing is learnt about NVLink; what the test does show is that the protocol runs on device tensors over the NCCL
backend and that handing the received rows and their offsets to `moe_experts` gives, bit for bit, what `moe_experts`
gives on the rows in place.  The multi-rank logic itself is covered on CPU (gloo, two ranks).  The work runs in a child
process with a time limit of its own: a rendezvous that cannot be set up on the box skips the test instead of holding
up the run.
"""
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import datetime
import torch
import torch.distributed as dist
from paper_2604_26881_b200 import binding as B, expert_parallel as EP, workloads as W

torch.cuda.set_device(0)
try:
    dist.init_process_group("nccl", rank=0, world_size=1, timeout=datetime.timedelta(seconds=60))
except Exception as e:                                   # no NCCL rendezvous on this box
    print("SKIP", repr(e)); sys.exit(0)
try:
    wl = W.MoEWorkload("ep1", T=200, H=256, E=12, I=128, k=3, Is=0, M=1, n_tenants=3, G=4, zipf_bias=True,
                       tenant_layout="uniform")
    wts = W.make_weights(wl, seed=5)
    x, tenant, mot = W.make_tokens(wl, seed=7)
    layer = B.MoELayer(H=wl.H, E=wl.E, I=wl.I, k=wl.k, Is=wl.Is, M=wl.M, n_tenants=wl.n_tenants, max_tokens=wl.T)
    layer.set_layer_weights(0, wts)
    layer.set_tables(slot_table=wts["slot_table"], model_of_tenant=mot)
    dev = layer.device
    T, k, H, E, R = wl.T, wl.k, wl.H, wl.E, wl.T * wl.k
    xd, td = x.to(dev), tenant.to(dev)
    i32 = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
    topk_idx, topk_w = i32(R), torch.zeros(R, dtype=torch.float32, device=dev)
    perm, inv_perm, expert_off, group_off = i32(R), i32(R), i32(E + 1), i32(E // wl.G + 1)
    x_perm = torch.zeros((R, H), dtype=torch.bfloat16, device=dev)
    B.moe_route(layer.ctx, 0, xd, td, T, topk_idx, topk_w)
    B.moe_dispatch(layer.ctx, xd, topk_idx, td, T, wl.G, perm, inv_perm, None, expert_off, group_off, x_perm)
    want = torch.zeros((R, H), dtype=torch.float32, device=dev)
    B.moe_experts(layer.ctx, 0, xd, x_perm, perm, expert_off, td, T, wl.G, want)
    torch.cuda.synchronize()

    calls = []
    def expert_step(rows, off):
        # the rows this rank received, sorted by expert, and their offsets: exactly what the library's call takes
        calls.append(int(rows.shape[0]))
        y = torch.zeros((rows.shape[0], H), dtype=torch.float32, device=dev)
        B.moe_experts(layer.ctx, 0, xd, rows.contiguous(), perm, off.to(torch.int32), td, T, wl.G, y)
        return y

    ep = EP.ExpertParallel([0] * E, expert_step)
    got = ep.forward_rows(x_perm, expert_off, H, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert B.moe_last_status(layer.ctx)[0] == 0
    assert calls == [R], calls
    assert torch.equal(got, want), float((got - want).abs().max())
    assert float(want.abs().max()) > 0
    layer.close()
    print("OK")
finally:
    dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def test_exchange_protocol_over_nccl_with_the_library_expert_step():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()), NCCL_NVLS_ENABLE="0")
    try:
        res = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=240)
    except subprocess.TimeoutExpired:
        pytest.skip("the NCCL rendezvous did not come up within the time limit on this box")
    out = res.stdout.strip().splitlines()
    if out and out[-1].startswith("SKIP"):
        pytest.skip(out[-1])
    assert res.returncode == 0 and out and out[-1] == "OK", res.stdout[-2000:] + res.stderr[-4000:]
