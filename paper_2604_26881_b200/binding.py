"""ctypes binding of libfaasmoe.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see
include/faasmoe.h) and passes raw device pointers of torch tensors.  Nothing is
computed in Python and there is no CPU fallback: if the library cannot be
loaded, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int, c_int32, c_int64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libfaasmoe.so")

MOE_OK = 0
MOE_ERR_NULL, MOE_ERR_SHAPE, MOE_ERR_G, MOE_ERR_STATE = -1, -2, -3, -4
MOE_ERR_CUDA, MOE_ERR_ALLOC, MOE_ERR_UNSUPPORTED = -5, -6, -7
MOE_DEV_BAD_TENANT, MOE_DEV_BAD_EXPERT, MOE_DEV_TIMEOUT = 1, 2, 8
MOE_OPT_EXPERT_PATH = 1
MOE_OPT_ROUTE_PATH = 2
MOE_OPT_PAIR_MODE = 3
MOE_OPT_WIDE_TILES = 4
MOE_OPT_TOKEN_MAJOR = 5
MOE_OPT_EARLY_SHARED = 6
MOE_OPT_EARLY_SHARED_SMS = 7
MOE_OPT_ROUTE_LANES = 8
MOE_OPT_DISPATCH_MODE = 9
MOE_OPT_BACKGROUND_LANES = 10
MOE_OPT_FUSED_DISPATCH = 11
MOE_OPT_HEAD_UNITS = 12
MOE_DISPATCH_SHARED, MOE_DISPATCH_PRIVATE = 0, 1
MOE_PATH_AUTO, MOE_PATH_FMA, MOE_PATH_TCGEN05 = 0, 1, 2

EXPORTS = ["moe_create", "moe_destroy", "moe_set_expert_pool", "moe_set_model_weights", "moe_set_slot_table",
           "moe_set_tenant_models", "moe_set_option", "moe_form_blocks", "moe_set_block_table", "moe_route", "moe_dispatch", "moe_experts", "moe_combine",
           "moe_layer_forward", "moe_residency_enable", "moe_layer_forward_paged", "moe_layer_forward_host", "moe_layer_forward_host_submit", "moe_layer_forward_host_wait", "moe_layer_forward_timed", "moe_stack_forward",
           "moe_get_workspace", "moe_last_status", "moe_last_plan", "moe_launch_count", "moe_strerror", "moe_dispatch_noalloc"]
MOE_DISPATCH_NOALLOC_MAX_WORDS = 1 << 18

STAGES = ["route", "dispatch", "plan", "experts_gateup", "experts_down", "combine"]


class MoeConfig(ctypes.Structure):
    _fields_ = [("hidden", c_int32), ("n_experts", c_int32), ("inter", c_int32), ("top_k", c_int32),
                ("shared_inter", c_int32), ("n_models", c_int32), ("n_tenants", c_int32), ("n_slots", c_int32),
                ("max_tokens", c_int32), ("n_layers", c_int32), ("rms_eps", c_float)]


class MoeError(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        super().__init__(f"{fn} failed with status {status}: {strerror(status)}")


_lib = None


def load_library(path: str | None = None):
    """Loads libfaasmoe.so (built in-tree by paper_2604_26881_b200.build).  Raises if missing."""
    global _lib
    if _lib is None:
        p = path or LIB_PATH
        if not os.path.exists(p):
            raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2604_26881_b200.build`")
        lib = ctypes.CDLL(p)
        for name in EXPORTS:
            getattr(lib, name)          # raises AttributeError if a symbol is missing
        lib.moe_strerror.restype = c_char_p
        lib.moe_strerror.argtypes = [c_int]
        lib.moe_launch_count.restype = c_int64
        lib.moe_launch_count.argtypes = [c_void_p]
        lib.moe_create.argtypes = [POINTER(MoeConfig), POINTER(c_void_p)]
        lib.moe_destroy.argtypes = [c_void_p]
        lib.moe_set_expert_pool.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p]
        lib.moe_set_model_weights.argtypes = [c_void_p, c_int, c_int] + [c_void_p] * 7
        lib.moe_set_slot_table.argtypes = [c_void_p, c_void_p]
        lib.moe_set_tenant_models.argtypes = [c_void_p, c_void_p]
        lib.moe_set_option.argtypes = [c_void_p, c_int, c_int]
        lib.moe_form_blocks.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p]
        lib.moe_set_block_table.argtypes = [c_void_p, c_void_p, c_int]
        lib.moe_route.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int] + [c_void_p] * 5
        lib.moe_dispatch.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int] + [c_void_p] * 7
        lib.moe_experts.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int,
                                    c_void_p, c_void_p, c_void_p]
        lib.moe_combine.argtypes = [c_void_p] + [c_void_p] * 5 + [c_int, c_void_p, c_void_p]
        lib.moe_layer_forward.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p]
        lib.moe_layer_forward_host.argtypes = lib.moe_layer_forward.argtypes
        lib.moe_layer_forward_host_submit.argtypes = lib.moe_layer_forward.argtypes + [POINTER(c_int64)]
        lib.moe_layer_forward_host_wait.argtypes = [c_void_p, c_int64]
        lib.moe_residency_enable.argtypes = [c_void_p, c_int] + [c_void_p] * 6
        lib.moe_layer_forward_paged.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_int, c_void_p,
                                                POINTER(c_int32), c_void_p]
        lib.moe_layer_forward_timed.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int, c_int, c_void_p,
                                                POINTER(c_float), c_void_p]
        lib.moe_stack_forward.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p]
        lib.moe_dispatch_noalloc.argtypes = [c_void_p] * 3 + [c_int] * 6 + [c_void_p] * 7
        lib.moe_get_workspace.argtypes = [c_void_p] + [POINTER(c_void_p)] * 8
        lib.moe_last_status.argtypes = [c_void_p, POINTER(c_int32), POINTER(c_int32)]
        lib.moe_last_plan.argtypes = [c_void_p, c_int, POINTER(c_int32)]
        _lib = lib
    return _lib


def strerror(status: int) -> str:
    return load_library().moe_strerror(int(status)).decode()


def _check(fn: str, status: int):
    if status != MOE_OK:
        raise MoeError(fn, status)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return c_void_p(t)
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream)


def moe_create(*, hidden, n_experts, inter, top_k, shared_inter=0, n_models=1, n_tenants=1, n_slots=None,
               max_tokens, n_layers=1, rms_eps=1e-6):
    cfg = MoeConfig(hidden, n_experts, inter, top_k, shared_inter, n_models, n_tenants,
                    n_slots if n_slots is not None else n_models * n_experts, max_tokens, n_layers, rms_eps)
    ctx = c_void_p()
    _check("moe_create", load_library().moe_create(byref(cfg), byref(ctx)))
    return ctx


def moe_destroy(ctx):
    _check("moe_destroy", load_library().moe_destroy(ctx))


def moe_set_expert_pool(ctx, layer, w_gate, w_up, w_down):
    _check("moe_set_expert_pool", load_library().moe_set_expert_pool(ctx, layer, _ptr(w_gate), _ptr(w_up), _ptr(w_down)))


def moe_set_model_weights(ctx, layer, model, router_w, router_bias=None, shared_gate_w=None, ws_gate=None, ws_up=None,
                          ws_down=None, rms_w=None):
    _check("moe_set_model_weights", load_library().moe_set_model_weights(
        ctx, layer, model, _ptr(router_w), _ptr(router_bias), _ptr(shared_gate_w), _ptr(ws_gate), _ptr(ws_up),
        _ptr(ws_down), _ptr(rms_w)))


def moe_set_slot_table(ctx, slot_host):
    assert slot_host.dtype == torch.int32 and not slot_host.is_cuda
    _check("moe_set_slot_table", load_library().moe_set_slot_table(ctx, _ptr(slot_host)))


def moe_set_tenant_models(ctx, model_of_tenant_host):
    assert model_of_tenant_host.dtype == torch.int32 and not model_of_tenant_host.is_cuda
    _check("moe_set_tenant_models", load_library().moe_set_tenant_models(ctx, _ptr(model_of_tenant_host)))


def moe_form_blocks(load, G):
    """Load-aware expert blocks from a host tensor load [M, E] (int64): returns block_of_expert [M, E] int32."""
    load = load.to(torch.int64).contiguous().cpu()
    M, E = load.shape
    out = torch.empty((M, E), dtype=torch.int32)
    _check("moe_form_blocks", load_library().moe_form_blocks(c_void_p(load.data_ptr()), M, E, G, c_void_p(out.data_ptr())))
    return out


def moe_set_block_table(ctx, block_of_expert, n_blocks=0):
    """block_of_expert: host int32 tensor [M, E] with ids in [0, n_blocks), or None for blocks of G consecutive experts."""
    if block_of_expert is None:
        _check("moe_set_block_table", load_library().moe_set_block_table(ctx, None, 0))
        return
    t = block_of_expert.to(torch.int32).contiguous().cpu()
    _check("moe_set_block_table", load_library().moe_set_block_table(ctx, c_void_p(t.data_ptr()), n_blocks))


def moe_set_option(ctx, option, value):
    _check("moe_set_option", load_library().moe_set_option(ctx, option, value))


def moe_route(ctx, layer, x, tenant_id, T, topk_idx, topk_w, shared_gate=None, tie_flag=None, stream=None):
    _check("moe_route", load_library().moe_route(ctx, layer, _ptr(x), _ptr(tenant_id), T, _ptr(topk_idx),
                                                 _ptr(topk_w), _ptr(shared_gate), _ptr(tie_flag), _stream(stream)))


def moe_dispatch(ctx, x, topk_idx, tenant_id, T, G, perm, inv_perm, tenant_expert_count=None, expert_off=None,
                 group_off=None, x_perm=None, stream=None):
    _check("moe_dispatch", load_library().moe_dispatch(
        ctx, _ptr(x), _ptr(topk_idx), _ptr(tenant_id), T, G, _ptr(perm), _ptr(inv_perm), _ptr(tenant_expert_count),
        _ptr(expert_off), _ptr(group_off), _ptr(x_perm), _stream(stream)))


def moe_dispatch_noalloc(topk_idx, tenant_id, model_of_tenant, T, k, E, M, n_tenants, G, perm, inv_perm,
                         tenant_expert_count=None, expert_off=None, group_off=None, status_out=None, stream=None):
    """moe_dispatch without a context and without any allocation inside the library: for callers that
    may not call cudaMalloc.  model_of_tenant is a DEVICE tensor here.  See include/faasmoe.h."""
    _check("moe_dispatch_noalloc", load_library().moe_dispatch_noalloc(
        _ptr(topk_idx), _ptr(tenant_id), _ptr(model_of_tenant), T, k, E, M, n_tenants, G, _ptr(perm), _ptr(inv_perm),
        _ptr(tenant_expert_count), _ptr(expert_off), _ptr(group_off), _ptr(status_out), _stream(stream)))


def moe_experts(ctx, layer, x, x_perm, perm, expert_off, tenant_id, T, G, y_perm, y_shared=None, stream=None):
    _check("moe_experts", load_library().moe_experts(ctx, layer, _ptr(x), _ptr(x_perm), _ptr(perm), _ptr(expert_off),
                                                     _ptr(tenant_id), T, G, _ptr(y_perm), _ptr(y_shared),
                                                     _stream(stream)))


def moe_combine(ctx, y_perm, inv_perm, topk_w, y_shared, shared_gate, T, out, stream=None):
    _check("moe_combine", load_library().moe_combine(ctx, _ptr(y_perm), _ptr(inv_perm), _ptr(topk_w), _ptr(y_shared),
                                                     _ptr(shared_gate), T, _ptr(out), _stream(stream)))


def moe_layer_forward_host_submit(ctx, layer, x_host, tenant_id_host, T, G, out_host, stream=None) -> int:
    """Enqueues H2D, the layer and D2H without waiting; returns the ticket to wait for (pinned host tensors)."""
    ticket = c_int64(-1)
    _check("moe_layer_forward_host_submit",
           load_library().moe_layer_forward_host_submit(ctx, layer, _ptr(x_host), _ptr(tenant_id_host), T, G, _ptr(out_host),
                                                        _stream(stream), byref(ticket)))
    return int(ticket.value)


def moe_layer_forward_host_wait(ctx, ticket: int):
    _check("moe_layer_forward_host_wait", load_library().moe_layer_forward_host_wait(ctx, ticket))


def moe_residency_enable(ctx, layer, host_gate, host_up, host_down, pool_gate, pool_up, pool_down):
    """host_*: CPU tensors [M*E, I, H] / [M*E, H, I] (pinned for asynchronous copies); pool_*: device tensors of n_slots slots."""
    _check("moe_residency_enable", load_library().moe_residency_enable(ctx, layer, _ptr(host_gate), _ptr(host_up),
                                                                       _ptr(host_down), _ptr(pool_gate), _ptr(pool_up),
                                                                       _ptr(pool_down)))


def moe_layer_forward_paged(ctx, layer, x, tenant_id, T, G, out, stream=None):
    """Returns (active experts, resident hits, experts loaded, experts evicted) of the call."""
    st = (c_int32 * 4)()
    _check("moe_layer_forward_paged", load_library().moe_layer_forward_paged(ctx, layer, _ptr(x), _ptr(tenant_id), T, G,
                                                                             _ptr(out), st, _stream(stream)))
    return int(st[0]), int(st[1]), int(st[2]), int(st[3])


def moe_layer_forward(ctx, layer, x, tenant_id, T, G, out, stream=None):
    _check("moe_layer_forward", load_library().moe_layer_forward(ctx, layer, _ptr(x), _ptr(tenant_id), T, G, _ptr(out),
                                                                 _stream(stream)))


def moe_layer_forward_host(ctx, layer, x_host, tenant_id_host, T, G, out_host, stream=None):
    assert not x_host.is_cuda and not tenant_id_host.is_cuda and not out_host.is_cuda
    _check("moe_layer_forward_host", load_library().moe_layer_forward_host(
        ctx, layer, _ptr(x_host), _ptr(tenant_id_host), T, G, _ptr(out_host), _stream(stream)))


def moe_layer_forward_timed(ctx, layer, x, tenant_id, T, G, out, stream=None):
    """One layer pass with CUDA events between the stages; returns {stage: ms}."""
    ms = (c_float * len(STAGES))()
    _check("moe_layer_forward_timed", load_library().moe_layer_forward_timed(
        ctx, layer, _ptr(x), _ptr(tenant_id), T, G, _ptr(out), ms, _stream(stream)))
    return {n: float(v) for n, v in zip(STAGES, ms)}


def moe_stage_times(ctx, x, tenant_id, T, G, out, reps=20, layer=0, stream=None):
    """Mean stage durations (ms) over `reps` timed passes."""
    acc = {n: 0.0 for n in STAGES}
    for _ in range(reps):
        for n, v in moe_layer_forward_timed(ctx, layer, x, tenant_id, T, G, out, stream).items():
            acc[n] += v
    return {n: v / reps for n, v in acc.items()}


def moe_stack_forward(ctx, x_inout, tenant_id, T, G, dbg_layer_inputs=None, dbg_layer_outputs=None, stream=None):
    _check("moe_stack_forward", load_library().moe_stack_forward(ctx, _ptr(x_inout), _ptr(tenant_id), T, G,
                                                                 _ptr(dbg_layer_inputs), _ptr(dbg_layer_outputs),
                                                                 _stream(stream)))


def moe_get_workspace(ctx):
    """Device addresses (ints) of the context's routing buffers of the last layer call."""
    names = ["topk_idx", "topk_w", "shared_gate", "tie_flag", "perm", "inv_perm", "expert_off", "group_off"]
    ptrs = [c_void_p() for _ in names]
    _check("moe_get_workspace", load_library().moe_get_workspace(ctx, *[byref(p) for p in ptrs]))
    return {n: p.value for n, p in zip(names, ptrs)}


class _DevicePointer:
    _TYPESTR = {torch.int32: "<i4", torch.float32: "<f4", torch.uint8: "|u1", torch.int16: "<i2"}

    def __init__(self, ptr, shape, dtype):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": self._TYPESTR[dtype],
                                         "data": (int(ptr), False), "version": 2}


def wrap_device_pointer(ptr: int, shape, dtype, device="cuda:0") -> torch.Tensor:
    """A torch view (no copy) of device memory owned by the library, e.g. a workspace buffer."""
    return torch.as_tensor(_DevicePointer(ptr, shape, dtype), device=device)


def moe_last_status(ctx):
    """(status bits, invocations, active experts); synchronises the device and clears the status."""
    st = c_int32(0)
    stats = (c_int32 * 2)()
    _check("moe_last_status", load_library().moe_last_status(ctx, byref(st), stats))
    return int(st.value), int(stats[0]), int(stats[1])


def moe_last_plan(ctx, T):
    """(routed tiles, shared-expert tiles, rows per tile) of the last expert call; synchronises the device."""
    plan = (c_int32 * 3)()
    _check("moe_last_plan", load_library().moe_last_plan(ctx, T, plan))
    return int(plan[0]), int(plan[1]), int(plan[2])


def moe_launch_count(ctx) -> int:
    return int(load_library().moe_launch_count(ctx))


class MoELayer:
    """Convenience holder: creates a context for a workload, uploads weights, keeps them alive."""

    def __init__(self, *, H, E, I, k, Is=0, M=1, n_tenants=1, max_tokens, n_layers=1, n_slots=None, rms_eps=1e-6,
                 device="cuda:0"):
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.H, self.E, self.I, self.k, self.Is, self.M = H, E, I, k, Is, M
        self.n_tenants, self.max_tokens, self.n_layers = n_tenants, max_tokens, n_layers
        self.ctx = moe_create(hidden=H, n_experts=E, inter=I, top_k=k, shared_inter=Is, n_models=M,
                              n_tenants=n_tenants, n_slots=n_slots, max_tokens=max_tokens, n_layers=n_layers,
                              rms_eps=rms_eps)
        self._keep = []

    def set_layer_weights(self, layer: int, wts: dict):
        """wts: tensors as produced by workloads.make_weights (CPU or CUDA); moved to the device and kept alive."""
        d = {k_: (v.to(self.device).contiguous() if v is not None else None) for k_, v in wts.items()
             if k_ != "slot_table"}
        self._keep.append(d)
        moe_set_expert_pool(self.ctx, layer, d["pool_gate"], d["pool_up"], d["pool_down"])
        for m in range(self.M):
            sel = lambda name: (d[name][m] if d.get(name) is not None else None)
            moe_set_model_weights(self.ctx, layer, m, sel("router_w"), sel("router_bias"), sel("shared_gate_w"),
                                  sel("ws_gate"), sel("ws_up"), sel("ws_down"), d.get("rms_w"))
        return d

    def set_tables(self, slot_table=None, model_of_tenant=None):
        if slot_table is not None:
            moe_set_slot_table(self.ctx, slot_table.to(torch.int32).cpu().contiguous())
        if model_of_tenant is not None:
            moe_set_tenant_models(self.ctx, model_of_tenant.to(torch.int32).cpu().contiguous())

    def close(self):
        if self.ctx is not None:
            moe_destroy(self.ctx)
            self.ctx = None
            self._keep.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
