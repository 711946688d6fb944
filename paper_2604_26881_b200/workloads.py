"""Seeded synthetic inputs for the multi-tenant MoE layer.

This module only draws random tensors and lays out ids; it contains none of
the layer's arithmetic.  Both the CUDA binding's tests and the CPU oracle's
tests take their inputs from here.

The shapes mirror the workload of the paper's evaluation (Sec. 4.2 / Sec. 5:
Qwen1.5-MoE-2.7B, 60 routed experts plus 4 shared experts per MoE layer,
several concurrent tenants) without using its trained weights or its
benchmark prompts: weights are bf16 N(0, 0.02), activations bf16 N(0, 1).
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class MoEWorkload:
    name: str
    T: int                 # tokens in the batch (ignored when ragged)
    H: int                 # hidden size
    E: int                 # routed experts per model
    I: int                 # intermediate size of one routed expert
    k: int                 # experts selected per token
    Is: int = 0            # intermediate size of the shared expert (0 = none)
    M: int = 1             # tenant models sharing the pool
    n_tenants: int = 1
    G: int = 1             # experts per expert block
    n_layers: int = 1
    zipf_bias: bool = False
    tenant_layout: str = "contiguous"   # contiguous | uniform | ragged
    rms_eps: float = 1e-6

    @property
    def n_slots(self) -> int:
        return self.M * self.E


QWEN = dict(H=2048, E=60, I=1408, k=4, Is=5632)

WORKLOADS = {
    # 64 tokens, 8 experts, top-2, no shared expert
    "tiny": MoEWorkload("tiny", T=64, H=256, E=8, I=128, k=2),
    # decode: 32 tokens from 4 tenants (8 each)
    "decode": MoEWorkload("decode", T=32, n_tenants=4, G=1, **QWEN),
    # prefill: 4096 tokens, Zipf-skewed expert load, 15 blocks of 4 experts
    "prefill": MoEWorkload("prefill", T=4096, n_tenants=1, G=4, zipf_bias=True, **QWEN),
    # 24 blocks, 16 tenants with ragged request lengths, 10 blocks of 6 experts
    "stack": MoEWorkload("stack", T=0, n_tenants=16, G=6, n_layers=24, tenant_layout="ragged", **QWEN),
    # 4 tenant models in one 240-slot routed pool (+4 shared experts)
    "pool": MoEWorkload("pool", T=2048, n_tenants=4, M=4, G=1, tenant_layout="uniform", **QWEN),
}


def scaled(w: MoEWorkload, **kw) -> MoEWorkload:
    """A copy of a workload with some fields replaced (smaller test cases)."""
    return replace(w, **kw)


def _gen(seed: int, *tags) -> torch.Generator:
    h = hashlib.sha256(repr((seed,) + tags).encode()).digest()
    g = torch.Generator(device="cpu")
    g.manual_seed(int.from_bytes(h[:8], "little") & 0x7FFFFFFFFFFFFFFF)
    return g


def _normal_bf16(shape, std, g) -> torch.Tensor:
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16)
    chunk = 1 << 26
    for i in range(0, n, chunk):
        m = min(chunk, n - i)
        out[i:i + m] = torch.empty(m, dtype=torch.float32).normal_(0.0, std, generator=g).to(torch.bfloat16)
    return out.view(*shape)


def zipf_router_bias(E: int, s: float, g: torch.Generator) -> torch.Tensor:
    """Per-expert logit bias: log of a Zipf(s) pmf over a seeded random ranking of the experts."""
    rank = torch.randperm(E, generator=g).to(torch.float64) + 1.0
    return (-s * torch.log(rank)).to(torch.float32)


def ragged_lengths(n_tenants: int, g: torch.Generator, mu=4.0, sigma=1.0, lo=1, hi=512):
    z = torch.empty(n_tenants, dtype=torch.float64).normal_(mu, sigma, generator=g)
    return [int(min(hi, max(lo, round(math.exp(v))))) for v in z.tolist()]


def make_weights(w: MoEWorkload, seed: int = 0, layer: int = 0, shuffle_slots: bool = False) -> dict:
    """CPU tensors of one layer: bf16 weights, f32 router bias, int32 slot table."""
    S = w.n_slots
    out = {
        "router_w": _normal_bf16((w.M, w.E, w.H), 0.02, _gen(seed, layer, "router_w")),
        "router_bias": None,
        "pool_gate": _normal_bf16((S, w.I, w.H), 0.02, _gen(seed, layer, "pool_gate")),
        "pool_up": _normal_bf16((S, w.I, w.H), 0.02, _gen(seed, layer, "pool_up")),
        "pool_down": _normal_bf16((S, w.H, w.I), 0.02, _gen(seed, layer, "pool_down")),
        "shared_gate_w": None, "ws_gate": None, "ws_up": None, "ws_down": None,
    }
    if w.zipf_bias:
        out["router_bias"] = torch.stack(
            [zipf_router_bias(w.E, 1.1, _gen(seed, layer, "router_bias", m)) for m in range(w.M)])
    if shuffle_slots:
        slot = torch.randperm(S, generator=_gen(seed, layer, "slot_table")).to(torch.int32)
    else:
        slot = torch.arange(S, dtype=torch.int32)
    out["slot_table"] = slot
    if w.Is > 0:
        out["shared_gate_w"] = _normal_bf16((w.M, w.H), 0.02, _gen(seed, layer, "shared_gate_w"))
        out["ws_gate"] = _normal_bf16((w.M, w.Is, w.H), 0.02, _gen(seed, layer, "ws_gate"))
        out["ws_up"] = _normal_bf16((w.M, w.Is, w.H), 0.02, _gen(seed, layer, "ws_up"))
        out["ws_down"] = _normal_bf16((w.M, w.H, w.Is), 0.02, _gen(seed, layer, "ws_down"))
    # RMSNorm scale of the stacked configuration: 1 + N(0, 0.02)
    out["rms_w"] = (1.0 + torch.empty(w.H, dtype=torch.float32).normal_(
        0.0, 0.02, generator=_gen(seed, layer, "rms_w"))).to(torch.bfloat16)
    return out


def make_tokens(w: MoEWorkload, seed: int = 0):
    """Returns x [T,H] bf16, tenant_id [T] int32, model_of_tenant [n_tenants] int32."""
    g = _gen(seed, "tokens", w.name)
    if w.tenant_layout == "ragged":
        lens = ragged_lengths(w.n_tenants, g)
        tenant = torch.cat([torch.full((n,), i, dtype=torch.int32) for i, n in enumerate(lens)])
    elif w.tenant_layout == "uniform":
        tenant = torch.randint(0, w.n_tenants, (w.T,), generator=g).to(torch.int32)
    else:
        per = -(-w.T // w.n_tenants)
        tenant = (torch.arange(w.T) // per).to(torch.int32)
    T = tenant.numel()
    x = _normal_bf16((T, w.H), 1.0, _gen(seed, "x", w.name))
    # tenants share models round-robin; with M == n_tenants each tenant has its own
    model_of_tenant = (torch.arange(w.n_tenants) % w.M).to(torch.int32)
    return x, tenant, model_of_tenant


def as_u16(t: torch.Tensor | None):
    """bf16 tensor -> numpy uint16 bit patterns (no copy of meaning, just a view)."""
    if t is None:
        return None
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def weights_as_numpy(wts: dict) -> dict:
    out = {}
    for key, v in wts.items():
        if v is None:
            out[key] = None
        elif v.dtype == torch.bfloat16:
            out[key] = as_u16(v)
        else:
            out[key] = v.contiguous().numpy()
    return out
