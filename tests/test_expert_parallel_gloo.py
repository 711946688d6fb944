"""Expert blocks placed on two ranks (CPU, gloo): every rank routes and dispatches its own tokens, rows travel to the rank
that holds their expert and their outputs travel back; the result must equal the single-process oracle of each rank's
batch.  The expert step here is a numpy SwiGLU on the exact bf16 weight values (the GPU library's call in production)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2604_26881_b200 import expert_parallel as EP
from paper_2604_26881_b200 import workloads as W


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _f64(u16):
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = W.MoEWorkload("ep", T=40 + 7 * rank, H=32, E=12, I=16, k=3, Is=16, M=1, n_tenants=3, G=4, zipf_bias=True,
                           tenant_layout="uniform")
        wts = W.make_weights(wl, seed=5)                      # the same weights on every rank
        wn = W.weights_as_numpy(wts)
        x, tenant, mot = W.make_tokens(wl, seed=100 + rank)   # its own batch
        xu, tn, mn = W.as_u16(x), tenant.numpy(), mot.numpy()
        ref = oracle.layer_forward(xu, tn, mn, wn, k=wl.k, G=wl.G)
        d = ref.dispatch
        # blocks of G experts placed by the rows they get (summed over the ranks), heaviest first
        nb = -(-wl.E // wl.G)
        rows = torch.tensor(np.diff(d.group_off).astype(np.int64))
        dist.all_reduce(rows)
        rank_of_block = EP.place_blocks(rows.tolist(), world)
        rank_of_expert = [rank_of_block[e // wl.G] for e in range(wl.E)]
        g64, u64, d64 = _f64(wn["pool_gate"]), _f64(wn["pool_up"]), _f64(wn["pool_down"])
        seen = []

        def expert_step(rows_x, expert_off):
            off = expert_off.tolist()
            y = np.zeros((rows_x.shape[0], wl.H))
            xr = rows_x.numpy()
            for e in range(wl.E):
                if off[e + 1] > off[e]:
                    assert rank_of_expert[e] == rank, "a rank only ever computes its own experts"
                    seen.append(e)
                    a = xr[off[e]:off[e + 1]]
                    gate = a @ g64[e].T
                    y[off[e]:off[e + 1]] = (gate / (1 + np.exp(-gate)) * (a @ u64[e].T)) @ d64[e].T
            return torch.from_numpy(y)

        ep = EP.ExpertParallel(rank_of_expert, expert_step)
        x_perm = torch.from_numpy(_f64(xu)[d.perm // wl.k])
        y_perm = ep.forward_rows(x_perm, torch.from_numpy(d.expert_off.astype(np.int64)), wl.H, out_dtype=torch.float64)
        np.testing.assert_allclose(y_perm.numpy(), ref.y_perm, rtol=1e-11, atol=1e-13)
        final = oracle.combine(y_perm.numpy(), d.inv_perm, ref.routing.topk_w, ref.y_shared, ref.routing.shared_gate)
        np.testing.assert_allclose(final, ref.out, rtol=1e-11, atol=1e-13)
        out[rank] = (rank_of_block, sorted(set(seen)), int(rows.sum()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_exchange_rows_and_match_the_oracle():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] and set(r0[0]) == {0, 1}            # the same placement on both ranks, both ranks used
    assert not set(r0[1]) & set(r1[1])                        # no expert computed on two ranks
    assert r0[2] == (40 + 47) * 3                             # every routed row of both batches was counted


def test_place_blocks_balances():
    # 10 -> rank 0, 9 -> rank 1, 8 -> the lighter rank 1 (17), then the two 1s -> rank 0 (11, 12): worked by hand
    assert EP.place_blocks([10, 1, 1, 9, 8], 2) == [0, 0, 0, 1, 1]
    rank_of = EP.place_blocks([10, 1, 1, 9, 8], 2)
    load = [sum(r for r, q in zip([10, 1, 1, 9, 8], rank_of) if q == k_) for k_ in range(2)]
    assert abs(load[0] - load[1]) <= 10 and sorted(set(rank_of)) == [0, 1]
    assert EP.place_blocks([5, 5, 5, 5], 4) == [0, 1, 2, 3]
