"""Thin ctypes binding of librr.so.  It only marshals arguments: every step of the
rectified MoE layer (routing, rectifications, expert FFN, combine, backward) runs in
the library's CUDA kernels.  PyTorch supplies device memory and streams.

There is no fallback: if librr.so is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

IR = 1
FR = 2
SCORE = 4   # a full expert drops its lowest scores instead of its latest tokens
LOCAL_CAP = 16  # capacity per (source group, expert): capacity/G slots each
FR_SOFTMAX = 8  # FR ranks nominees by softmax value instead of raw logit (needs FR)
GRAD_EXACT = 1
BF16 = 0
F32 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librr.so")

_TABLE_FIELDS = ["topk_expert", "route_slot", "slot_token", "slot_rank", "drop_count", "ir_expert",
                 "ir_pos", "ir_offset", "ir_token", "expert_count", "n_routed", "row_offset",
                 "row_token", "row_weight", "token_rows", "combine_w"]


class _CTables(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _TABLE_FIELDS]


class _CShape(C.Structure):
    _fields_ = [("T", C.c_int32), ("E", C.c_int32), ("k", C.c_int32), ("capacity", C.c_int32),
                ("G", C.c_int32), ("d", C.c_int32), ("d_ff", C.c_int32), ("dtype", C.c_int32),
                ("mode", C.c_uint32), ("flags", C.c_uint32), ("trace", C.c_void_p)]


class RRError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (rr_status {code})")


_lib = None


def lib():
    """Loads librr.so; raises if it has not been built (python -m paper_2402_12399_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with paper_2402_12399_b200/build.py; "
                              "there is no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        L.rr_status_string.restype = C.c_char_p
        L.rr_status_string.argtypes = [C.c_int]
        L.rr_route_workspace_bytes.argtypes = [C.c_int] * 5 + [C.c_uint, C.POINTER(C.c_size_t)]
        L.rr_route.argtypes = [C.c_void_p] + [C.c_int] * 5 + [C.c_uint, C.POINTER(_CTables), C.c_void_p,
                                                             C.c_size_t, C.c_void_p]
        L.rr_route_noalloc.argtypes = [C.c_void_p] + [C.c_int] * 5 + [C.c_uint, C.POINTER(_CTables), C.c_void_p,
                                                                     C.c_void_p]
        L.rr_moe_workspace_bytes.argtypes = [C.POINTER(_CShape)] + [C.POINTER(C.c_size_t)] * 3
        L.rr_moe_fwd.argtypes = [C.POINTER(_CShape)] + [C.c_void_p] * 5 + [C.POINTER(_CTables)] + \
            [C.c_void_p] * 3 + [C.c_size_t, C.c_void_p]
        L.rr_moe_bwd.argtypes = [C.POINTER(_CShape)] + [C.c_void_p] * 6 + [C.POINTER(_CTables)] + \
            [C.c_void_p] * 7 + [C.c_size_t, C.c_void_p]
        L.rr_check.argtypes = [C.c_void_p, C.c_void_p]
        L.rr_test_set_wait_limit_ns.argtypes = [C.c_ulonglong]
        L.rr_test_set_wait_limit_ns.restype = None
        L.rr_gate_workspace_bytes.argtypes = [C.c_int] * 3 + [C.POINTER(C.c_size_t)] * 2
        L.rr_gate_fwd.argtypes = [C.c_int] * 4 + [C.c_void_p] * 4 + [C.c_size_t, C.c_void_p]
        L.rr_gate_bwd.argtypes = [C.c_int] * 4 + [C.c_void_p] * 6 + [C.c_size_t, C.c_void_p]
        L.rr_gate_route_workspace_bytes.argtypes = [C.c_int] * 5 + [C.c_uint, C.c_int, C.POINTER(C.c_size_t)]
        L.rr_gate_route.argtypes = [C.c_int] * 5 + [C.c_uint, C.c_int, C.c_int] + [C.c_void_p] * 3 + [C.POINTER(_CTables), C.c_float] + \
            [C.c_void_p] * 4 + [C.c_size_t, C.c_void_p]
        L.rr_route_loss_workspace_bytes.argtypes = [C.c_int] * 5 + [C.c_uint, C.POINTER(C.c_size_t)]
        L.rr_route_loss.argtypes = [C.c_void_p] + [C.c_int] * 5 + [C.c_uint, C.POINTER(_CTables), C.c_float] + [C.c_void_p] * 4 + \
            [C.c_size_t, C.c_void_p]
        L.rr_aux_workspace_bytes.argtypes = [C.c_int] * 2 + [C.POINTER(C.c_size_t)]
        L.rr_aux_loss_fwd.argtypes = [C.c_int] * 3 + [C.c_void_p] * 2 + [C.c_float] + [C.c_void_p] * 4 + \
            [C.c_size_t, C.c_void_p]
        L.rr_aux_loss_bwd.argtypes = [C.c_int] * 2 + [C.c_void_p] * 2 + [C.c_float] * 2 + [C.c_int, C.c_void_p,
                                                                                             C.c_void_p]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().rr_status_string(code).decode()


def _ok(code, where):
    if code != 0:
        raise RRError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class RouteTables:
    """Device tensors of the routing result; meanings as documented in include/rr.h."""
    T: int
    E: int
    k: int
    capacity: int
    G: int
    mode: int
    topk_expert: torch.Tensor
    route_slot: torch.Tensor
    slot_token: torch.Tensor
    slot_rank: torch.Tensor
    drop_count: torch.Tensor
    ir_expert: torch.Tensor
    ir_pos: torch.Tensor
    ir_offset: torch.Tensor
    ir_token: torch.Tensor
    expert_count: torch.Tensor
    n_routed: torch.Tensor
    row_offset: torch.Tensor
    row_token: torch.Tensor
    row_weight: torch.Tensor
    token_rows: torch.Tensor
    combine_w: torch.Tensor

    def c_struct(self):
        # storage pointer, not data_ptr(): an empty table (capacity 0, T 0) still has a real address
        def addr(t):
            return t.untyped_storage().data_ptr() + t.storage_offset() * t.element_size()
        return _CTables(*[addr(getattr(self, n)) for n in _TABLE_FIELDS])


def alloc_tables(T, E, k, capacity, G, mode, device="cuda") -> RouteTables:
    i32 = dict(dtype=torch.int32, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    capacity_ = max(capacity, 0)
    R = E * capacity_ + T
    # +4 elements so that empty tables still own an aligned, non-null pointer
    def buf(n, **kw):
        n = max(n, 0)
        return torch.empty(n + 4, **kw)[:n]
    return RouteTables(
        T, E, k, capacity, G, mode,
        topk_expert=buf(T * (k + 1), **i32).view(T, k + 1),
        route_slot=buf(T * (k + 1), **i32).view(T, k + 1),
        slot_token=buf(E * capacity_, **i32).view(E, capacity_),
        slot_rank=buf(E * capacity_, dtype=torch.int8, device=device).view(E, capacity_),
        drop_count=buf(T, **i32), ir_expert=buf(T, **i32), ir_pos=buf(T, **i32),
        ir_offset=buf(E + 1, **i32), ir_token=buf(T, **i32), expert_count=buf(E, **i32),
        n_routed=buf(E, **i32), row_offset=buf(E + 1, **i32), row_token=buf(R, **i32),
        row_weight=buf(R, **f32), token_rows=buf(T * (k + 2), **i32).view(T, k + 2),
        combine_w=buf(T * (k + 2), **f32).view(T, k + 2))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A zero-filled workspace (the status word in its header must start at zero)."""
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def route_workspace_bytes(T, E, k, capacity, G, mode) -> int:
    n = C.c_size_t(0)
    _ok(lib().rr_route_workspace_bytes(T, E, k, capacity, G, mode, C.byref(n)), "rr_route_workspace_bytes")
    return n.value


def route(logits: torch.Tensor, k: int, capacity: int, G: int, mode: int, tables: RouteTables | None = None,
          workspace: torch.Tensor | None = None) -> RouteTables:
    """rr_route on a [T,E] fp32 CUDA tensor; asynchronous on the current stream."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    T, E = logits.shape
    if workspace is None:
        workspace = alloc_workspace(route_workspace_bytes(T, E, k, capacity, G, mode), logits.device)
    if tables is None:
        tables = alloc_tables(T, E, k, capacity, G, mode, logits.device)
    cs = tables.c_struct()
    _ok(lib().rr_route(_ptr(logits), T, E, k, capacity, G, mode, C.byref(cs), _ptr(workspace),
                       workspace.numel(), _stream()), "rr_route")
    tables._workspace = workspace
    return tables


def route_loss_workspace_bytes(T, E, k, capacity, G, mode) -> int:
    n = C.c_size_t(0)
    _ok(lib().rr_route_loss_workspace_bytes(T, E, k, capacity, G, mode, C.byref(n)), "rr_route_loss_workspace_bytes")
    return n.value


def route_loss(logits: torch.Tensor, k: int, capacity: int, G: int, mode: int, alpha: float,
               tables: RouteTables | None = None, workspace: torch.Tensor | None = None, aux=None):
    """rr_route_loss: routing and the load-balance loss in the one routing kernel.
    Returns (tables, (loss [1], f [E], P [E]))."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    T, E = logits.shape
    if workspace is None:
        workspace = alloc_workspace(route_loss_workspace_bytes(T, E, k, capacity, G, mode), logits.device)
    if tables is None:
        tables = alloc_tables(T, E, k, capacity, G, mode, logits.device)
    if aux is None:
        aux = (torch.empty(1, dtype=torch.float32, device=logits.device),
               torch.empty(E, dtype=torch.float32, device=logits.device),
               torch.empty(E, dtype=torch.float32, device=logits.device))
    cs = tables.c_struct()
    _ok(lib().rr_route_loss(_ptr(logits), T, E, k, capacity, G, mode, C.byref(cs), alpha, _ptr(aux[0]), _ptr(aux[1]),
                            _ptr(aux[2]), _ptr(workspace), workspace.numel(), _stream()), "rr_route_loss")
    tables._workspace = workspace
    return tables, aux


def route_noalloc(logits: torch.Tensor, k: int, capacity: int, G: int, mode: int, tables: RouteTables,
                  status: torch.Tensor | None = None) -> RouteTables:
    """rr_route_noalloc: routing whose scratch is a fixed array inside librr.so, for callers that
    cannot allocate device memory.  `tables` (and the optional zero-filled `status` word) are the
    caller's; the call itself allocates nothing.  Overlapping calls on one GPU race on the array."""
    T, E = logits.shape
    cs = tables.c_struct()
    _ok(lib().rr_route_noalloc(_ptr(logits), T, E, k, capacity, G, mode, C.byref(cs), _ptr(status), _stream()),
        "rr_route_noalloc")
    return tables


def test_set_wait_limit_ns(ns: int) -> None:
    """Testing aid: time limit of the waits a test can make run out (0 restores the 2 s of production)."""
    lib().rr_test_set_wait_limit_ns(int(ns))


def check(workspace: torch.Tensor) -> None:
    """Synchronises the current stream and raises if the device latched an error."""
    _ok(lib().rr_check(_ptr(workspace), _stream()), "rr_check")


def _shape(T, E, k, capacity, G, d, d_ff, dtype, mode, flags=0, trace=None):
    s = _CShape(T, E, k, capacity, G, d, d_ff, dtype, mode, flags, None)
    if trace is not None:
        s._trace_keepalive = trace
        s.trace = C.cast(trace, C.c_void_p)
    return s


class Trace:
    """Eight CUDA events the library records around its kernels (see rr_moe_shape.trace)."""

    def __init__(self):
        self.events = [torch.cuda.Event(enable_timing=True) for _ in range(8)]
        for e in self.events:
            e.record()          # events are created lazily; recording gives them a handle
        torch.cuda.synchronize()
        self.array = (C.c_void_p * 8)(*[e.cuda_event for e in self.events])

    def ms(self, i, j):
        return self.events[i].elapsed_time(self.events[j])


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"hidden/weights must be bfloat16 or float32, got {t.dtype}")


def moe_workspace_bytes(T, E, k, capacity, G, d, d_ff, dtype, mode, flags=0):
    """(fwd workspace bytes, bwd workspace bytes, saved bytes)."""
    s = _shape(T, E, k, capacity, G, d, d_ff, dtype, mode, flags)
    a, b, c = C.c_size_t(0), C.c_size_t(0), C.c_size_t(0)
    _ok(lib().rr_moe_workspace_bytes(C.byref(s), C.byref(a), C.byref(b), C.byref(c)), "rr_moe_workspace_bytes")
    return a.value, b.value, c.value


def moe_fwd(hidden, W1, W3, W2, logits, tables: RouteTables, out=None, saved=None, workspace=None,
            trace: "Trace | None" = None):
    """rr_moe_fwd; returns out [T,d] fp32.  Pass `saved` (see moe_workspace_bytes) when training."""
    T, d = hidden.shape
    E, d_ff, _ = W1.shape
    dt = _dtype_code(hidden)
    for w in (W1, W3, W2):
        assert w.is_cuda and w.is_contiguous() and _dtype_code(w) == dt
    s = _shape(T, E, tables.k, tables.capacity, tables.G, d, d_ff, dt, tables.mode,
               trace=None if trace is None else trace.array)
    if workspace is None:
        workspace = alloc_workspace(moe_workspace_bytes(T, E, tables.k, tables.capacity, tables.G, d, d_ff, dt,
                                                        tables.mode)[0], hidden.device)
    if out is None:
        out = torch.empty(T, d, dtype=torch.float32, device=hidden.device)
    cs = tables.c_struct()
    _ok(lib().rr_moe_fwd(C.byref(s), _ptr(hidden), _ptr(W1), _ptr(W3), _ptr(W2), _ptr(logits), C.byref(cs),
                         _ptr(out), _ptr(saved), _ptr(workspace), workspace.numel(), _stream()), "rr_moe_fwd")
    out._workspace = workspace
    return out


def moe_bwd(dout, hidden, W1, W3, W2, logits, tables: RouteTables, saved, grad_exact=False, workspace=None,
            grads=None, trace: "Trace | None" = None):
    """rr_moe_bwd; returns (dhidden, dlogits, dW1, dW3, dW2), all fp32."""
    T, d = hidden.shape
    E, d_ff, _ = W1.shape
    dt = _dtype_code(hidden)
    flags = GRAD_EXACT if grad_exact else 0
    s = _shape(T, E, tables.k, tables.capacity, tables.G, d, d_ff, dt, tables.mode, flags,
               trace=None if trace is None else trace.array)
    if workspace is None:
        workspace = alloc_workspace(moe_workspace_bytes(T, E, tables.k, tables.capacity, tables.G, d, d_ff, dt,
                                                        tables.mode, flags)[1], hidden.device)
    if grads is None:
        f32 = dict(dtype=torch.float32, device=hidden.device)
        grads = (torch.empty(T, d, **f32), torch.empty(T, E, **f32), torch.empty(E, d_ff, d, **f32),
                 torch.empty(E, d_ff, d, **f32), torch.empty(E, d, d_ff, **f32))
    dh, dl, dW1, dW3, dW2 = grads
    cs = tables.c_struct()
    _ok(lib().rr_moe_bwd(C.byref(s), _ptr(dout), _ptr(hidden), _ptr(W1), _ptr(W3), _ptr(W2), _ptr(logits),
                         C.byref(cs), _ptr(saved), _ptr(dh), _ptr(dl), _ptr(dW1), _ptr(dW3), _ptr(dW2),
                         _ptr(workspace), workspace.numel(), _stream()), "rr_moe_bwd")
    dh._workspace = workspace
    return grads


def gate_workspace_bytes(T, E, d):
    """(fwd workspace bytes, bwd workspace bytes) of the gate projection."""
    a, b = C.c_size_t(0), C.c_size_t(0)
    _ok(lib().rr_gate_workspace_bytes(T, E, d, C.byref(a), C.byref(b)), "rr_gate_workspace_bytes")
    return a.value, b.value


def gate_fwd(hidden: torch.Tensor, Wg: torch.Tensor, logits: torch.Tensor | None = None,
             workspace: torch.Tensor | None = None) -> torch.Tensor:
    """rr_gate_fwd; returns logits [T,E] fp32 = hidden . Wg^T."""
    T, d = hidden.shape
    E = Wg.shape[0]
    dt = _dtype_code(hidden)
    assert Wg.is_cuda and Wg.is_contiguous() and _dtype_code(Wg) == dt and Wg.shape[1] == d
    if workspace is None:
        workspace = alloc_workspace(gate_workspace_bytes(T, E, d)[0], hidden.device)
    if logits is None:
        logits = torch.empty(T, E, dtype=torch.float32, device=hidden.device)
    _ok(lib().rr_gate_fwd(T, E, d, dt, _ptr(hidden), _ptr(Wg), _ptr(logits), _ptr(workspace), workspace.numel(),
                          _stream()), "rr_gate_fwd")
    logits._workspace = workspace
    return logits


def gate_route_workspace_bytes(T, E, k, capacity, G, mode, d) -> int:
    n = C.c_size_t(0)
    _ok(lib().rr_gate_route_workspace_bytes(T, E, k, capacity, G, mode, d, C.byref(n)), "rr_gate_route_workspace_bytes")
    return n.value


def gate_route(hidden: torch.Tensor, Wg: torch.Tensor, k: int, capacity: int, G: int, mode: int, alpha: float | None = None,
               logits: torch.Tensor | None = None, tables: RouteTables | None = None, workspace: torch.Tensor | None = None,
               aux=None):
    """rr_gate_route: gate projection, routing and (with `alpha`) the load-balance loss in two launches;
    the selection is made in the projection's epilogue.  Returns (logits, tables, (loss, f, P) or None)."""
    T, d = hidden.shape
    E = Wg.shape[0]
    dt = _dtype_code(hidden)
    assert Wg.is_cuda and Wg.is_contiguous() and _dtype_code(Wg) == dt and Wg.shape[1] == d
    if workspace is None:
        workspace = alloc_workspace(gate_route_workspace_bytes(T, E, k, capacity, G, mode, d), hidden.device)
    if logits is None:
        logits = torch.empty(T, E, dtype=torch.float32, device=hidden.device)
    if tables is None:
        tables = alloc_tables(T, E, k, capacity, G, mode, hidden.device)
    if alpha is not None and aux is None:
        aux = (torch.empty(1, dtype=torch.float32, device=hidden.device),
               torch.empty(E, dtype=torch.float32, device=hidden.device),
               torch.empty(E, dtype=torch.float32, device=hidden.device))
    cs = tables.c_struct()
    a = aux if alpha is not None else (None, None, None)
    _ok(lib().rr_gate_route(T, E, k, capacity, G, mode, d, dt, _ptr(hidden), _ptr(Wg), _ptr(logits), C.byref(cs),
                            0.0 if alpha is None else alpha, _ptr(a[0]), _ptr(a[1]), _ptr(a[2]), _ptr(workspace),
                            workspace.numel(), _stream()), "rr_gate_route")
    tables._workspace = workspace
    logits._workspace = workspace
    return logits, tables, (aux if alpha is not None else None)


def gate_bwd(dlogits: torch.Tensor, hidden: torch.Tensor, Wg: torch.Tensor, dhidden: torch.Tensor,
             dWg: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """rr_gate_bwd; ADDS dlogits . Wg to `dhidden` in place and returns dWg [E,d] fp32."""
    T, d = hidden.shape
    E = Wg.shape[0]
    dt = _dtype_code(hidden)
    assert dlogits.dtype == torch.float32 and dlogits.is_contiguous() and dlogits.shape == (T, E)
    assert dhidden.dtype == torch.float32 and dhidden.is_contiguous() and dhidden.shape == (T, d)
    if workspace is None:
        workspace = alloc_workspace(gate_workspace_bytes(T, E, d)[1], hidden.device)
    if dWg is None:
        dWg = torch.empty(E, d, dtype=torch.float32, device=hidden.device)
    _ok(lib().rr_gate_bwd(T, E, d, dt, _ptr(dlogits), _ptr(hidden), _ptr(Wg), _ptr(dWg), _ptr(dhidden),
                          _ptr(workspace), workspace.numel(), _stream()), "rr_gate_bwd")
    return dWg


def aux_workspace_bytes(T, E):
    """Workspace bytes of the load-balance loss."""
    a = C.c_size_t(0)
    _ok(lib().rr_aux_workspace_bytes(T, E, C.byref(a)), "rr_aux_workspace_bytes")
    return a.value


def aux_loss_fwd(logits: torch.Tensor, topk_expert: torch.Tensor, alpha: float,
                 workspace: torch.Tensor | None = None):
    """rr_aux_loss_fwd; returns (loss [1], f [E], P [E]) fp32 on the device.  `topk_expert` is the
    routing table [T,k+1] (or any int32 [T,n] whose column 0 is the first choice)."""
    T, E = logits.shape
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    assert topk_expert.dtype == torch.int32 and topk_expert.is_contiguous() and topk_expert.shape[0] == T
    if workspace is None:
        workspace = alloc_workspace(aux_workspace_bytes(T, E), logits.device)
    loss = torch.empty(1, dtype=torch.float32, device=logits.device)
    f = torch.empty(E, dtype=torch.float32, device=logits.device)
    P = torch.empty(E, dtype=torch.float32, device=logits.device)
    stride = topk_expert.shape[1] if topk_expert.dim() == 2 else 1
    _ok(lib().rr_aux_loss_fwd(T, E, stride, _ptr(logits), _ptr(topk_expert), alpha, _ptr(loss), _ptr(f), _ptr(P),
                              _ptr(workspace), workspace.numel(), _stream()), "rr_aux_loss_fwd")
    loss._workspace = workspace
    return loss, f, P


def aux_loss_bwd(logits: torch.Tensor, f: torch.Tensor, alpha: float, scale: float = 1.0,
                 dlogits: torch.Tensor | None = None, accumulate: bool = False) -> torch.Tensor:
    """rr_aux_loss_bwd; writes (or, with accumulate, adds) dL/da [T,E] into `dlogits` and returns it."""
    T, E = logits.shape
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    assert f.dtype == torch.float32 and f.is_contiguous() and f.numel() == E
    if dlogits is None:
        assert not accumulate
        dlogits = torch.empty(T, E, dtype=torch.float32, device=logits.device)
    assert dlogits.dtype == torch.float32 and dlogits.is_contiguous() and dlogits.shape == (T, E)
    _ok(lib().rr_aux_loss_bwd(T, E, _ptr(logits), _ptr(f), alpha, scale, int(accumulate), _ptr(dlogits), _stream()),
        "rr_aux_loss_bwd")
    return dlogits
