"""TEST INFRASTRUCTURE ONLY: ctypes front-end of the fp64 CPU oracle (moe_oracle.c).

The oracle states what the FaaSMoE MoE layer computes (gating and top-k,
Sec. 2.1; micro-batched dispatch into expert blocks, Sec. 3 / Sec. 4.1; expert
execution; aggregation, Sec. 3) in plain C loops over doubles.  It is
independent of the CUDA library: nothing here imports the GPU package and the
GPU package never imports this.  Only tests, the smoke check and the
CPU-baseline leg of the benchmark may use it.

All array arguments are numpy arrays; bf16 tensors are passed as ``uint16``
bit patterns.  Parity status: every function below is pinned by the CPU tests
(brute force, closed forms, library restatements, invariants); the paper's own
resource figures (CPU %, GB) are not reproducible here: parity unpinned for
those, and they are not computed by this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile moe_oracle.c with gcc (plain -O2, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
        for name in ("oracle_route", "oracle_dispatch", "oracle_experts", "oracle_shared_expert",
                     "oracle_combine", "oracle_rmsnorm", "oracle_invocations", "oracle_form_blocks",
                     "oracle_invocations_table"):
            getattr(_lib, name).restype = ctypes.c_int
        _lib.oracle_round_bf16.restype = None
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError(f"expected {dtype}, got {a.dtype}")
    return a


@dataclass
class Routing:
    probs: np.ndarray        # [T,E] f64
    topk_idx: np.ndarray     # [T,k] i32
    topk_w: np.ndarray       # [T,k] f64
    shared_gate: np.ndarray  # [T] f64
    tie_flag: np.ndarray     # [T] u8


@dataclass
class Dispatch:
    perm: np.ndarray                 # [T*k] i32
    inv_perm: np.ndarray             # [T*k] i32
    tenant_expert_count: np.ndarray  # [n_tenants,E] i32
    expert_off: np.ndarray           # [M*E+1] i32
    group_off: np.ndarray            # [M*ceil(E/G)+1] i32
    n_invocations: int


def route(x, tenant_id, model_of_tenant, router_w, router_bias=None, shared_gate_w=None, *, k):
    """Gating network + top-k (Sec. 2.1).  x [T,H] u16; router_w [M,E,H] u16."""
    lib = _load()
    x = _c(x, np.uint16); tenant_id = _c(tenant_id, np.int32)
    model_of_tenant = _c(model_of_tenant, np.int32)
    router_w = _c(router_w, np.uint16); router_bias = _c(router_bias, np.float32)
    shared_gate_w = _c(shared_gate_w, np.uint16)
    T, H = x.shape
    M, E, H2 = router_w.shape
    assert H2 == H and 1 <= k <= E
    probs = np.empty((T, E), np.float64)
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    sg = np.empty((T,), np.float64)
    flag = np.empty((T,), np.uint8)
    rc = lib.oracle_route(_p(x), _p(tenant_id), T, H, E, k, M, len(model_of_tenant), _p(model_of_tenant),
                          _p(router_w), _p(router_bias), _p(shared_gate_w),
                          _p(probs), _p(idx), _p(w), _p(sg), _p(flag))
    if rc != 0:
        raise ValueError(f"oracle_route failed: {rc}")
    return Routing(probs, idx, w, sg, flag)


def dispatch(topk_idx, tenant_id, model_of_tenant, *, n_models, E, G):
    """Micro-batched routing requests per expert block (Sec. 3, Sec. 4.1)."""
    lib = _load()
    topk_idx = _c(topk_idx, np.int32); tenant_id = _c(tenant_id, np.int32)
    model_of_tenant = _c(model_of_tenant, np.int32)
    T, k = topk_idx.shape
    n_tenants = len(model_of_tenant)
    if not (1 <= G <= E):
        raise ValueError("G out of range")
    B = (E + G - 1) // G
    perm = np.empty((T * k,), np.int32)
    inv = np.empty((T * k,), np.int32)
    cnt = np.empty((n_tenants, E), np.int32)
    eoff = np.empty((n_models * E + 1,), np.int32)
    goff = np.empty((n_models * B + 1,), np.int32)
    ninv = ctypes.c_int32(0)
    rc = lib.oracle_dispatch(_p(topk_idx), _p(tenant_id), T, E, k, n_models, n_tenants, _p(model_of_tenant), G,
                             _p(perm), _p(inv), _p(cnt), _p(eoff), _p(goff), ctypes.byref(ninv))
    if rc != 0:
        raise ValueError(f"oracle_dispatch failed: {rc}")
    return Dispatch(perm, inv, cnt, eoff, goff, int(ninv.value))


SHARED, PRIVATE = 0, 1


@dataclass
class Invocations:
    n_invocations: int
    tenant_invocations: np.ndarray   # [n_tenants] i32
    token_fanout: np.ndarray         # [T] i32
    n_row_batches: int


def invocations(topk_idx, tenant_id, model_of_tenant, *, n_models, E, G, mode, batch_rows=128):
    """Invocations of expert blocks under a shared orchestrator (mode SHARED: rows of all tenants to a block travel
    together) or private ones (mode PRIVATE: every tenant batches only its own tokens) -- Sec. 4.2, Sec. 5."""
    lib = _load()
    topk_idx = _c(topk_idx, np.int32); tenant_id = _c(tenant_id, np.int32)
    model_of_tenant = _c(model_of_tenant, np.int32)
    T, k = topk_idx.shape
    n_tenants = len(model_of_tenant)
    ninv, nbatch = ctypes.c_int32(0), ctypes.c_int32(0)
    per_tenant = np.empty((n_tenants,), np.int32)
    fan = np.empty((T,), np.int32)
    rc = lib.oracle_invocations(_p(topk_idx), _p(tenant_id), T, E, k, n_models, n_tenants, _p(model_of_tenant), G, mode,
                                batch_rows, ctypes.byref(ninv), _p(per_tenant), _p(fan), ctypes.byref(nbatch))
    if rc != 0:
        raise ValueError(f"oracle_invocations failed: {rc}")
    return Invocations(int(ninv.value), per_tenant, fan, int(nbatch.value))


def form_blocks(load, *, G):
    """Load-aware expert blocks (Sec. 5): experts in order of (load descending, id ascending), each to the least
    loaded block that still has room.  load [M,E] -> block_of_expert [M,E] int32 with ids in [0, ceil(E/G))."""
    lib = _load()
    load = np.ascontiguousarray(load, dtype=np.int64)
    M, E = load.shape
    out = np.empty((M, E), np.int32)
    rc = lib.oracle_form_blocks(_p(load), M, E, G, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_form_blocks failed: {rc}")
    return out


@dataclass
class TableInvocations:
    n_invocations: int
    tenant_invocations: np.ndarray   # [n_tenants] i32
    token_fanout: np.ndarray         # [T] i32
    block_rows: np.ndarray           # [M, n_blocks] i32


def invocations_table(topk_idx, tenant_id, model_of_tenant, block_of_expert, *, n_blocks, mode):
    """Invocation accounting when the blocks are given by a table [M,E] instead of ranges of G experts."""
    lib = _load()
    topk_idx = _c(topk_idx, np.int32); tenant_id = _c(tenant_id, np.int32)
    model_of_tenant = _c(model_of_tenant, np.int32); block_of_expert = _c(block_of_expert, np.int32)
    T, k = topk_idx.shape
    M, E = block_of_expert.shape
    n_tenants = len(model_of_tenant)
    ninv = ctypes.c_int32(0)
    per_tenant = np.empty((n_tenants,), np.int32); fan = np.empty((T,), np.int32)
    rows = np.empty((M, n_blocks), np.int32)
    rc = lib.oracle_invocations_table(_p(topk_idx), _p(tenant_id), T, E, k, M, n_tenants, _p(model_of_tenant),
                                      _p(block_of_expert), n_blocks, mode, ctypes.byref(ninv), _p(per_tenant), _p(fan),
                                      _p(rows))
    if rc != 0:
        raise ValueError(f"oracle_invocations_table failed: {rc}")
    return TableInvocations(int(ninv.value), per_tenant, fan, rows)


def residency_lru(active_sets, n_slots):
    """On-demand residency of experts in a fixed number of device slots (the scale-to-zero idea of the abstract and
    Sec. 3 applied to device memory): every expert is parked until a batch routes to it.

    For every batch, in order: the experts it needs that are resident are hits; every missing one, in ascending id,
    takes a free slot (lowest index) or else evicts the resident expert that was needed longest ago among those the
    current batch does not need (ties: lowest slot index).  Returns a list of (hits, loads, evictions, slot_of) per
    batch, slot_of a dict expert -> slot after the batch.  Raises if a batch needs more experts than there are slots.
    """
    owner = [-1] * n_slots
    history = []                                     # the batches so far, as sets
    out = []
    for step, need in enumerate(active_sets):
        need = sorted(set(int(e) for e in need))
        if len(need) > n_slots:
            raise ValueError("more active experts than slots")

        def last_needed(e):                          # latest earlier batch that needed expert e
            for back in range(len(history) - 1, -1, -1):
                if e in history[back]:
                    return back
            return -1
        hits = sum(1 for e in need if e in owner)
        loads = evictions = 0
        for e in need:
            if e in owner:
                continue
            if -1 in owner:
                slot = owner.index(-1)
            else:
                cand = [s for s in range(n_slots) if owner[s] not in need]
                slot = min(cand, key=lambda s: (last_needed(owner[s]), s))
                evictions += 1
            owner[slot] = e
            loads += 1
        history.append(set(need))
        out.append((hits, loads, evictions, {e: s for s, e in enumerate(owner) if e >= 0}))
    return out


def experts(x, tenant_id, topk_idx, perm, model_of_tenant, pool_gate, pool_up, pool_down, slot_table, *, n_models):
    """SwiGLU FFN of the activated experts over the routed rows, in segment order (Sec. 3)."""
    lib = _load()
    x = _c(x, np.uint16); tenant_id = _c(tenant_id, np.int32); topk_idx = _c(topk_idx, np.int32)
    perm = _c(perm, np.int32); model_of_tenant = _c(model_of_tenant, np.int32)
    pool_gate = _c(pool_gate, np.uint16); pool_up = _c(pool_up, np.uint16); pool_down = _c(pool_down, np.uint16)
    slot_table = _c(slot_table, np.int32)
    T, H = x.shape
    k = topk_idx.shape[1]
    S, I, H2 = pool_gate.shape
    assert H2 == H and pool_up.shape == (S, I, H) and pool_down.shape == (S, H, I)
    E = len(slot_table) // n_models
    y = np.empty((T * k, H), np.float64)
    rc = lib.oracle_experts(_p(x), _p(tenant_id), _p(topk_idx), _p(perm), T, H, E, I, k, n_models,
                            _p(model_of_tenant), _p(pool_gate), _p(pool_up), _p(pool_down), S, _p(slot_table), _p(y))
    if rc != 0:
        raise ValueError(f"oracle_experts failed: {rc}")
    return y


def shared_expert(x, tenant_id, model_of_tenant, ws_gate, ws_up, ws_down):
    """The always-active shared expert (Sec. 5), ungated.  ws_gate [M,Is,H] u16."""
    lib = _load()
    x = _c(x, np.uint16); tenant_id = _c(tenant_id, np.int32); model_of_tenant = _c(model_of_tenant, np.int32)
    ws_gate = _c(ws_gate, np.uint16); ws_up = _c(ws_up, np.uint16); ws_down = _c(ws_down, np.uint16)
    T, H = x.shape
    M, Is, H2 = ws_gate.shape
    assert H2 == H and ws_up.shape == (M, Is, H) and ws_down.shape == (M, H, Is)
    y = np.empty((T, H), np.float64)
    rc = lib.oracle_shared_expert(_p(x), _p(tenant_id), T, H, Is, M, _p(model_of_tenant),
                                  _p(ws_gate), _p(ws_up), _p(ws_down), _p(y))
    if rc != 0:
        raise ValueError(f"oracle_shared_expert failed: {rc}")
    return y


def combine(y_perm, inv_perm, topk_w, y_shared=None, shared_gate=None):
    """Weighted aggregation per token (Sec. 3)."""
    lib = _load()
    y_perm = _c(y_perm, np.float64); inv_perm = _c(inv_perm, np.int32); topk_w = _c(topk_w, np.float64)
    y_shared = _c(y_shared, np.float64); shared_gate = _c(shared_gate, np.float64)
    T, k = topk_w.shape
    H = y_perm.shape[1]
    out = np.empty((T, H), np.float64)
    rc = lib.oracle_combine(_p(y_perm), _p(inv_perm), _p(topk_w), _p(y_shared),
                            _p(shared_gate) if y_shared is not None else None, T, H, k, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_combine failed: {rc}")
    return out


def rmsnorm(x, g, eps):
    lib = _load()
    x = _c(x, np.uint16); g = _c(g, np.uint16)
    T, H = x.shape
    xn = np.empty((T, H), np.float64)
    lib.oracle_rmsnorm(_p(x), _p(g), T, H, ctypes.c_double(eps), _p(xn))
    return xn


def round_bf16(v):
    """fp64 -> bf16 bit patterns, one round-to-nearest-even step."""
    lib = _load()
    v = _c(v, np.float64)
    out = np.empty(v.shape, np.uint16)
    lib.oracle_round_bf16(_p(v), ctypes.c_size_t(v.size), _p(out))
    return out


@dataclass
class LayerResult:
    routing: Routing
    dispatch: Dispatch
    y_perm: np.ndarray            # [T*k,H] f64
    y_shared: np.ndarray | None   # [T,H] f64
    out: np.ndarray               # [T,H] f64


def layer_forward(x, tenant_id, model_of_tenant, weights, *, k, G, topk_override=None):
    """Whole MoE layer: gate -> dispatch -> experts -> aggregate (Sec. 3).

    ``weights`` is a mapping with router_w [M,E,H], optional router_bias [M,E],
    pool_gate/pool_up/pool_down, slot_table [M*E], and optionally
    shared_gate_w [M,H], ws_gate/ws_up/ws_down.  ``topk_override`` (idx [T,k],
    rows mask [T]) replaces the selection of the masked tokens: the test
    protocol for tokens whose ranks are closer than fp32 can resolve.
    """
    M, E, _ = weights["router_w"].shape
    has_shared = weights.get("ws_gate") is not None
    r = route(x, tenant_id, model_of_tenant, weights["router_w"], weights.get("router_bias"),
              weights.get("shared_gate_w") if has_shared else None, k=k)
    if topk_override is not None:
        idx_o, mask = topk_override
        idx = r.topk_idx.copy()
        w = r.topk_w.copy()
        for t in np.nonzero(mask)[0]:
            idx[t] = idx_o[t]
            w[t] = r.probs[t, idx_o[t]]
        r = Routing(r.probs, idx, w, r.shared_gate, r.tie_flag)
    d = dispatch(r.topk_idx, tenant_id, model_of_tenant, n_models=M, E=E, G=G)
    y = experts(x, tenant_id, r.topk_idx, d.perm, model_of_tenant, weights["pool_gate"], weights["pool_up"],
                weights["pool_down"], weights["slot_table"], n_models=M)
    ys = None
    if has_shared:
        ys = shared_expert(x, tenant_id, model_of_tenant, weights["ws_gate"], weights["ws_up"], weights["ws_down"])
    out = combine(y, d.inv_perm, r.topk_w, ys, r.shared_gate if has_shared else None)
    return LayerResult(r, d, y, ys, out)


def block_forward(x, tenant_id, model_of_tenant, weights, *, k, G, eps, xn_override=None, topk_override=None):
    """One block of the stacked configuration: RMSNorm -> MoE layer -> residual add.

    x [T,H] u16.  Returns (x_next u16, xn u16, LayerResult).  xn is rounded to
    bf16 before the layer, and the residual stream is rounded to bf16 after the
    add.  ``xn_override`` substitutes the normalised input (teacher forcing).
    """
    xn = round_bf16(rmsnorm(x, weights["rms_w"], eps)) if xn_override is None else xn_override
    res = layer_forward(xn, tenant_id, model_of_tenant, weights, k=k, G=G, topk_override=topk_override)
    xf = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    x_next = round_bf16(xf + res.out)
    return x_next, xn, res
