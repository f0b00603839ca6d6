"""ctypes front end of the CPU oracle (``rr_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

The oracle restates, in plain fp64 C, what one rectified MoE layer computes
(arXiv 2402.12399: Section 3 Eq. 1-2, Section 4.1 Eq. 3, Section 4.2,
Appendix A Eq. 6).  Nothing in the CUDA library or its Python binding may import
this module; it exists so that tests, the smoke check and the benchmark's CPU
baseline can compare against an independent statement of the method.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rr_oracle.c")
_LIB = os.path.join(_HERE, "librr_oracle.so")

IR = 1
FR = 2
SCORE = 4   # a full expert drops its lowest scores (the other reading of Section 3), not its latest tokens
FR_SOFTMAX = 8  # FR ranks nominees by the fixed fp32 softmax value instead of the raw logit (needs FR)
LOCAL_CAP = 16  # capacity per (source group, expert): C/G slots each (needs G | C)
F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile rr_oracle.c with gcc (no fast-math, no contraction) if needed."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def num_threads() -> int:
    return int(lib().rro_num_threads())


def set_num_threads(n: int) -> None:
    lib().rro_set_num_threads(C.c_int(n))


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class Tables:
    """Routing result; field meanings are given at ``rro_route`` in rr_oracle.c."""
    T: int
    E: int
    k: int
    C: int
    G: int
    mode: int
    topk_expert: np.ndarray
    route_slot: np.ndarray
    slot_token: np.ndarray
    slot_rank: np.ndarray
    drop_count: np.ndarray
    ir_expert: np.ndarray
    ir_pos: np.ndarray
    ir_offset: np.ndarray
    ir_token: np.ndarray
    expert_count: np.ndarray
    n_routed: np.ndarray
    row_offset: np.ndarray
    row_token: np.ndarray
    row_weight: np.ndarray
    token_rows: np.ndarray
    combine_w: np.ndarray


class OracleError(ValueError):
    pass


_ERR = {1: "invalid argument", 2: "non-finite logit", 3: "out of memory"}


def _check(rc):
    if rc != 0:
        raise OracleError(_ERR.get(rc, f"error {rc}"))


def route(logits: np.ndarray, k: int, capacity: int, G: int, mode: int) -> Tables:
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, E = logits.shape
    Cc = int(capacity)
    t = Tables(
        T, E, k, Cc, G, mode,
        topk_expert=np.empty((T, k + 1), np.int32),
        route_slot=np.empty((T, k + 1), np.int32),
        slot_token=np.empty((E, max(Cc, 0)), np.int32),
        slot_rank=np.empty((E, max(Cc, 0)), np.int8),
        drop_count=np.empty(T, np.int32),
        ir_expert=np.empty(T, np.int32),
        ir_pos=np.empty(T, np.int32),
        ir_offset=np.empty(E + 1, np.int32),
        ir_token=np.empty(T, np.int32),
        expert_count=np.empty(E, np.int32),
        n_routed=np.empty(E, np.int32),
        row_offset=np.empty(E + 1, np.int32),
        row_token=np.empty(E * max(Cc, 0) + T, np.int32),
        row_weight=np.empty(E * max(Cc, 0) + T, np.float64),
        token_rows=np.empty((T, k + 2), np.int32),
        combine_w=np.empty((T, k + 2), np.float64),
    )
    rc = lib().rro_route(
        _p(logits), C.c_int(T), C.c_int(E), C.c_int(k), C.c_int(Cc), C.c_int(G), C.c_uint(mode),
        _p(t.topk_expert), _p(t.route_slot), _p(t.slot_token), _p(t.slot_rank), _p(t.drop_count),
        _p(t.ir_expert), _p(t.ir_pos), _p(t.ir_offset), _p(t.ir_token), _p(t.expert_count),
        _p(t.n_routed), _p(t.row_offset), _p(t.row_token), _p(t.row_weight), _p(t.token_rows),
        _p(t.combine_w))
    _check(rc)
    return t


def softmax32(row: np.ndarray) -> np.ndarray:
    """The fixed single-precision softmax of one row of logits (``rro_softmax32``)."""
    row = np.ascontiguousarray(row, dtype=np.float32)
    g = np.empty_like(row)
    lib().rro_softmax32(_p(row), C.c_int(row.shape[0]), _p(g))
    return g


def weights(logits: np.ndarray, t: Tables) -> np.ndarray:
    """Combine weights for frozen routing tables and (possibly perturbed) logits."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    w = np.empty((t.T, t.k + 2), np.float64)
    _check(lib().rro_weights(_p(logits), C.c_int(t.T), C.c_int(t.E), C.c_int(t.k),
                             _p(t.topk_expert), _p(t.route_slot), _p(t.drop_count),
                             _p(t.ir_expert), _p(w)))
    return w


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16  # raw bf16 bit patterns
    raise TypeError(f"oracle tensors are float32 or uint16 (bf16 bits), got {a.dtype}")


def _same_dtype(*arrs):
    codes = {_dtype_code(a) for a in arrs}
    if len(codes) != 1:
        raise TypeError("hidden, weights and dout must share one element type")
    return codes.pop()


def forward_tokens(hidden, W1, W3, W2, logits, t: Tables, tokens=None, want_rows=False):
    """out_i (fp64) for the listed tokens (all if None); optionally the raw E_e(x_i) rows."""
    dt = _same_dtype(hidden, W1, W3, W2)
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    d = hidden.shape[1]
    d_ff = W1.shape[1]
    tokens = np.arange(t.T, dtype=np.int32) if tokens is None else np.ascontiguousarray(tokens, np.int32)
    out = np.empty((len(tokens), d), np.float64)
    y = np.empty((len(tokens), t.k + 2, d), np.float64) if want_rows else None
    _check(lib().rro_forward_tokens(
        _p(hidden), _p(W1), _p(W3), _p(W2), C.c_int(dt), _p(logits), C.c_int(t.T), C.c_int(t.E),
        C.c_int(t.k), C.c_int(d), C.c_int(d_ff), _p(t.topk_expert), _p(t.route_slot),
        _p(t.drop_count), _p(t.ir_expert), _p(tokens), C.c_int(len(tokens)), _p(out), _p(y)))
    return (out, y) if want_rows else out


def backward_tokens(hidden, W1, W3, W2, dout, logits, t: Tables, tokens=None, grad_exact=False):
    """(dhidden_i, dlogits_i) in fp64 for the listed tokens (all if None)."""
    dt = _same_dtype(hidden, W1, W3, W2, dout)
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    d = hidden.shape[1]
    d_ff = W1.shape[1]
    tokens = np.arange(t.T, dtype=np.int32) if tokens is None else np.ascontiguousarray(tokens, np.int32)
    dh = np.empty((len(tokens), d), np.float64)
    dl = np.empty((len(tokens), t.E), np.float64)
    _check(lib().rro_backward_tokens(
        _p(hidden), _p(W1), _p(W3), _p(W2), _p(dout), C.c_int(dt), _p(logits), C.c_int(t.T),
        C.c_int(t.E), C.c_int(t.k), C.c_int(d), C.c_int(d_ff), C.c_int(1 if grad_exact else 0),
        _p(t.topk_expert), _p(t.route_slot), _p(t.drop_count), _p(t.ir_expert), _p(tokens),
        C.c_int(len(tokens)), _p(dh), _p(dl)))
    return dh, dl


def backward_expert(hidden, W1, W3, W2, dout, t: Tables, e: int):
    """(dW1_e, dW3_e, dW2_e) in fp64 for one expert, summed over all its live rows."""
    dt = _same_dtype(hidden, W1, W3, W2, dout)
    d = hidden.shape[1]
    d_ff = W1.shape[1]
    dW1 = np.empty((d_ff, d), np.float64)
    dW3 = np.empty((d_ff, d), np.float64)
    dW2 = np.empty((d, d_ff), np.float64)
    _check(lib().rro_backward_expert(
        _p(hidden), _p(W1), _p(W3), _p(W2), _p(dout), C.c_int(dt), C.c_int(e), C.c_int(d),
        C.c_int(d_ff), _p(t.row_offset), _p(t.row_token), _p(t.row_weight), _p(dW1), _p(dW3),
        _p(dW2)))
    return dW1, dW3, dW2


def backward_expert_cols(hidden, W1, W3, W2, dout, t: Tables, e: int, cols):
    """Rows `cols` of dW1_e, dW3_e ([n,d]) and columns `cols` of dW2_e ([d,n]) in fp64."""
    dt = _same_dtype(hidden, W1, W3, W2, dout)
    d = hidden.shape[1]
    d_ff = W1.shape[1]
    cols = np.ascontiguousarray(cols, np.int32)
    n = len(cols)
    dW1 = np.empty((n, d), np.float64)
    dW3 = np.empty((n, d), np.float64)
    dW2 = np.empty((d, n), np.float64)
    _check(lib().rro_backward_expert_cols(
        _p(hidden), _p(W1), _p(W3), _p(W2), _p(dout), C.c_int(dt), C.c_int(e), C.c_int(d),
        C.c_int(d_ff), _p(t.row_offset), _p(t.row_token), _p(t.row_weight), _p(cols), C.c_int(n),
        _p(dW1), _p(dW3), _p(dW2)))
    return dW1, dW3, dW2


def gate_fwd(hidden: np.ndarray, Wg: np.ndarray) -> np.ndarray:
    """a[T,E] (fp64) = hidden[T,d] . Wg[E,d]^T  (Eq. 1)."""
    dt = _same_dtype(hidden, Wg)
    T, d = hidden.shape
    E = Wg.shape[0]
    out = np.empty((T, E), np.float64)
    _check(lib().rro_gate_fwd(_p(hidden), _p(Wg), C.c_int(dt), C.c_int(T), C.c_int(E), C.c_int(d), _p(out)))
    return out


def gate_bwd(dlogits: np.ndarray, hidden: np.ndarray, Wg: np.ndarray):
    """(dWg[E,d], dhidden[T,d]) in fp64 for given dL/da[T,E]."""
    dt = _same_dtype(hidden, Wg)
    T, d = hidden.shape
    E = Wg.shape[0]
    dl = np.ascontiguousarray(dlogits, np.float64)
    dWg, dh = np.empty((E, d), np.float64), np.empty((T, d), np.float64)
    _check(lib().rro_gate_bwd(_p(dl), _p(hidden), _p(Wg), C.c_int(dt), C.c_int(T), C.c_int(E), C.c_int(d),
                              _p(dWg), _p(dh)))
    return dWg, dh


def aux_loss(logits: np.ndarray, topk_expert: np.ndarray, alpha: float):
    """(L, f[E], P[E]) of the load-balance loss L = alpha E sum_e f_e P_e (Section 5.1): f from the
    first choices (column 0 of topk_expert, before capacity), P the mean softmax over all experts."""
    a = np.ascontiguousarray(logits, np.float32)
    te = np.ascontiguousarray(topk_expert, np.int32)
    T, E = a.shape
    loss = C.c_double(0.0)
    f, P = np.empty(E, np.float64), np.empty(E, np.float64)
    _check(lib().rro_aux_loss(_p(a), _p(te), C.c_int(te.shape[1]), C.c_int(T), C.c_int(E), C.c_double(alpha),
                              C.byref(loss), _p(f), _p(P)))
    return loss.value, f, P


def aux_loss_bwd(logits: np.ndarray, f: np.ndarray, alpha: float, scale: float = 1.0) -> np.ndarray:
    """dL/da [T,E] (fp64) with the counts f held constant."""
    a = np.ascontiguousarray(logits, np.float32)
    T, E = a.shape
    ff = np.ascontiguousarray(f, np.float64)
    out = np.empty((T, E), np.float64)
    _check(lib().rro_aux_loss_bwd(_p(a), _p(ff), C.c_int(T), C.c_int(E), C.c_double(alpha), C.c_double(scale),
                                  _p(out)))
    return out
