"""ctypes front end of the CPU oracle (``cstep_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()``
and by the ``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``. The
product package never imports this module and this module never imports the
product package.

Arrays are numpy, on the host. Every call works on a list of tensors
(``w`` and optional ``lam`` per tensor) and returns freshly allocated outputs.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cstep_oracle.c")
_LIB = os.path.join(_HERE, "libcstep_oracle.so")

FUSE_FP16, FUSE_LAMBDA, FUSE_PENALTY, FUSE_BF16, FUSE_E4M3, FUSE_E5M2 = 1, 2, 4, 8, 16, 32
CRITERIA = {"l2": 0, "l1": 1, "max": 2}

CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
          "-fno-unsafe-math-optimizations", "-Wall"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.run(["gcc"] + CFLAGS + ["-o", tmp, _SRC, "-lm"], check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Tensor(C.Structure):
    _fields_ = [("w", C.c_void_p), ("lam", C.c_void_p), ("theta", C.c_void_p),
                ("mask", C.c_void_p), ("lam_out", C.c_void_p), ("grad", C.c_void_p),
                ("theta_h", C.c_void_p), ("numel", C.c_int64), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 4)]


class _Result(C.Structure):
    _fields_ = [("n_units", C.c_int64), ("n_zero", C.c_int64), ("n_keep", C.c_int64),
                ("tau_key", C.c_uint64), ("tau_id", C.c_int64), ("n_gt", C.c_int64),
                ("n_tie", C.c_int64), ("n_tie_kept", C.c_int64), ("tau_norm", C.c_float)]


class _Spec(C.Structure):
    _fields_ = [("kind", C.c_int32), ("kinds", C.c_int32), ("nd", C.c_int32), ("crit", C.c_int32),
                ("bs", C.c_int64 * 4)]


class _OptTensor(C.Structure):
    _fields_ = [("w", C.c_void_p), ("theta", C.c_void_p), ("lam", C.c_void_p), ("grad", C.c_void_p),
                ("buf1", C.c_void_p), ("buf2", C.c_void_p), ("numel", C.c_int64)]


class _Opt(C.Structure):
    _fields_ = [("kind", C.c_int32), ("lr", C.c_float), ("momentum", C.c_float),
                ("weight_decay", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("step", C.c_int64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        assert L.orc_sizeof_tensor() == C.sizeof(_Tensor)
        assert L.orc_sizeof_result() == C.sizeof(_Result)
        L.orc_round_count.restype = C.c_int64
        L.orc_round_count.argtypes = [C.c_double, C.c_int64]
        L.orc_f32_to_f16.restype = C.c_uint16
        L.orc_f32_to_f16.argtypes = [C.c_uint32]
        L.orc_f16_to_f32.restype = C.c_uint32
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_f16_array.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_f32_to_bf16_array.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_f32_to_bf16_range.argtypes = [C.c_uint32, C.c_int64, C.c_void_p]
        L.orc_f32_to_f16_range.argtypes = [C.c_uint32, C.c_int64, C.c_void_p]
        L.orc_form_u.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_int64, C.c_void_p]
        L.orc_lagrange.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_uint,
                                   C.c_int64, C.c_void_p, C.c_void_p]
        L.orc_structure_norms.restype = C.c_int64
        L.orc_structure_norms.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_int, C.c_int,
                                          C.c_int, C.c_void_p]
        L.orc_cstep_prune.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_float, C.c_uint,
                                      C.c_void_p]
        L.orc_cstep_filter.argtypes = list(L.orc_cstep_prune.argtypes)
        L.orc_cstep_structure.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_float, C.c_int, C.c_uint,
                                          C.c_void_p]
        L.orc_cstep_block.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_float, C.c_int,
                                      C.c_int, C.c_uint, C.c_void_p]
        L.orc_cstep_quantize.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_uint]
        assert L.orc_sizeof_spec() == C.sizeof(_Spec)
        L.orc_structure_values.restype = C.c_int64
        L.orc_structure_values.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_void_p, C.c_void_p]
        L.orc_cstep_structured.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_float, C.c_void_p, C.c_uint,
                                           C.c_void_p]
        L.orc_f32_to_fp8.restype = C.c_uint8
        L.orc_f32_to_fp8.argtypes = [C.c_uint32, C.c_int]
        L.orc_fp8_to_f32.restype = C.c_uint32
        L.orc_fp8_to_f32.argtypes = [C.c_uint8, C.c_int]
        L.orc_f32_to_fp8_array.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p]
        L.orc_f32_to_fp8_range.argtypes = [C.c_uint32, C.c_int64, C.c_int, C.c_void_p]
        L.orc_lagrange_update.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_uint]
        assert L.orc_sizeof_opt_tensor() == C.sizeof(_OptTensor) and L.orc_sizeof_opt() == C.sizeof(_Opt)
        L.orc_lstep_update.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_void_p]
        if not L.orc_denormals_ok():
            raise RuntimeError("subnormal fp32 arithmetic is flushed in this process; "
                               "the oracle's results would not be IEEE")
        _lib = L
    return _lib


@dataclass
class Result:
    n_units: int
    n_zero: int
    n_keep: int
    tau_key: int
    tau_id: int
    n_gt: int
    n_tie: int
    n_tie_kept: int
    tau_norm: float


@dataclass
class Outputs:
    theta: List[np.ndarray]
    mask: List[np.ndarray]
    lam: List[np.ndarray]        # multipliers after the call (copy of the input if not updated)
    grad: List[np.ndarray]
    theta_h: List[np.ndarray]
    result: Optional[Result] = None


def fuse_bits(fuse: Sequence[str]) -> int:
    table = {"fp16": FUSE_FP16, "lambda": FUSE_LAMBDA, "penalty": FUSE_PENALTY, "bf16": FUSE_BF16,
             "e4m3": FUSE_E4M3, "e5m2": FUSE_E5M2}
    b = 0
    for f in fuse:
        b |= table[f]
    return b


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _table(ws, lams, thetas=None):
    T = len(ws)
    keep = []          # keeps every numpy buffer alive while the C call runs
    tab = (_Tensor * max(T, 1))()
    out = Outputs([], [], [], [], [])
    for t in range(T):
        w = np.ascontiguousarray(ws[t], dtype=np.float32)
        lam = None if (lams is None or lams[t] is None) else np.ascontiguousarray(
            lams[t], dtype=np.float32)
        n = w.size
        theta = (np.empty(w.shape, np.float32) if thetas is None
                 else np.ascontiguousarray(thetas[t], dtype=np.float32).copy())
        mask = np.empty(w.shape, np.uint8)
        lam_out = np.zeros(w.shape, np.float32)
        grad = np.zeros(w.shape, np.float32)
        theta_h = np.zeros(w.shape, np.uint16)
        keep += [w, lam]
        e = tab[t]
        e.w, e.lam, e.theta, e.mask = _ptr(w), _ptr(lam), _ptr(theta), _ptr(mask)
        e.lam_out, e.grad, e.theta_h = _ptr(lam_out), _ptr(grad), _ptr(theta_h)
        e.numel, e.ndim = n, w.ndim
        assert 1 <= w.ndim <= 4
        for d in range(4):
            e.shape[d] = w.shape[d] if d < w.ndim else 1
        out.theta.append(theta); out.mask.append(mask); out.lam.append(lam_out)
        out.grad.append(grad); out.theta_h.append(theta_h)
    return tab, out, keep


def _result(r: _Result) -> Result:
    return Result(r.n_units, r.n_zero, r.n_keep, r.tau_key, r.tau_id, r.n_gt, r.n_tie,
                  r.n_tie_kept, float(r.tau_norm))


def round_count(s: float, n: int) -> int:
    return int(lib().orc_round_count(float(s), int(n)))


def form_u(w: np.ndarray, lam: Optional[np.ndarray], mu: float) -> np.ndarray:
    w = np.ascontiguousarray(w, dtype=np.float32)
    u = np.empty_like(w)
    l = None if lam is None else np.ascontiguousarray(lam, dtype=np.float32)
    lib().orc_form_u(_ptr(w), _ptr(l), C.c_float(mu), w.size, _ptr(u))
    return u


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """binary16 bits (uint16) of each fp32 value (or uint32 bit pattern) in x."""
    b = np.ascontiguousarray(x)
    if b.dtype == np.float32:
        b = b.view(np.uint32)
    assert b.dtype == np.uint32
    out = np.empty(b.shape, np.uint16)
    lib().orc_f32_to_f16_array(_ptr(b), b.size, _ptr(out))
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(x)
    if b.dtype == np.float32:
        b = b.view(np.uint32)
    assert b.dtype == np.uint32
    out = np.empty(b.shape, np.uint16)
    lib().orc_f32_to_bf16_array(_ptr(b), b.size, _ptr(out))
    return out


def f32_to_bf16_range(first: int, n: int) -> np.ndarray:
    out = np.empty(n, np.uint16)
    lib().orc_f32_to_bf16_range(C.c_uint32(first), n, _ptr(out))
    return out


def f32_to_f16_range(first: int, n: int) -> np.ndarray:
    out = np.empty(n, np.uint16)
    lib().orc_f32_to_f16_range(C.c_uint32(first), n, _ptr(out))
    return out


def f16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, np.uint32)
    L = lib()
    flat_h, flat_o = h.reshape(-1), out.reshape(-1)
    for i in range(flat_h.size):
        flat_o[i] = L.orc_f16_to_f32(int(flat_h[i]))
    return out.view(np.float32)


FP8_FORMATS = {"e4m3": 0, "e5m2": 1}


def f32_to_fp8_bits(x: np.ndarray, fmt: str) -> np.ndarray:
    """8-bit code (uint8) of each fp32 value (or uint32 bit pattern) in x; fmt 'e4m3' or 'e5m2'."""
    b = np.ascontiguousarray(x)
    if b.dtype == np.float32:
        b = b.view(np.uint32)
    assert b.dtype == np.uint32
    out = np.empty(b.shape, np.uint8)
    lib().orc_f32_to_fp8_array(_ptr(b), b.size, FP8_FORMATS[fmt], _ptr(out))
    return out


def f32_to_fp8_range(first: int, n: int, fmt: str) -> np.ndarray:
    out = np.empty(n, np.uint8)
    lib().orc_f32_to_fp8_range(C.c_uint32(first), n, FP8_FORMATS[fmt], _ptr(out))
    return out


def fp8_bits_to_f32(h: np.ndarray, fmt: str) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint8)
    L = lib()
    out = np.array([L.orc_fp8_to_f32(int(v), FP8_FORMATS[fmt]) for v in h.reshape(-1)], np.uint32)
    return out.view(np.float32).reshape(h.shape)


def _spec(kind: str, block=None, criterion: str = "l2") -> _Spec:
    """kind: 'filter', 'neuron', 'structure' (filters and neurons) or 'block' with
    ``block`` = the block extents, one per tensor dimension."""
    sp = _Spec()
    sp.crit = CRITERIA[criterion]
    if kind == "block":
        sp.kind, sp.nd = 1, len(block)
        for d, b in enumerate(block):
            sp.bs[d] = int(b)
    else:
        sp.kind, sp.kinds = 0, {"filter": 1, "neuron": 2, "structure": 3}[kind]
    return sp


def structure_values(ws, lams, mu: float, kind: str, block=None, criterion: str = "l2") -> np.ndarray:
    """The fp64 value every ranked structure is ranked by, in global structure order."""
    tab, _, keep = _table(ws, lams)
    sp = _spec(kind, block, criterion)
    S = lib().orc_structure_values(tab, len(ws), C.c_float(mu), C.byref(sp), None)
    nu = np.empty(S, np.float64)
    lib().orc_structure_values(tab, len(ws), C.c_float(mu), C.byref(sp), _ptr(nu))
    return nu


def cstep_structured(ws, lams, s: float, mu: float, kind: str, block=None, criterion: str = "l2",
                     fuse: Sequence[str] = ()) -> Outputs:
    """Structured pruning by a specification: leading-index slices or n-D blocks, ranked by the
    L2, L1 or max criterion."""
    tab, out, keep = _table(ws, lams)
    r = _Result()
    sp = _spec(kind, block, criterion)
    rc = lib().orc_cstep_structured(tab, len(ws), float(s), C.c_float(mu), C.byref(sp), fuse_bits(fuse), C.byref(r))
    assert rc == 0, rc
    out.result = _result(r)
    return out


def structure_norms(ws, lams, mu: float, kind: str, block=(4, 4)) -> np.ndarray:
    """fp64 nu of every ranked structure, in global structure order."""
    tab, _, keep = _table(ws, lams)
    k = {"filter": 0, "neuron": 0, "structure": 0, "block": 1}[kind]
    bh = {"filter": 1, "neuron": 2, "structure": 3}.get(kind, block[0])
    S = lib().orc_structure_norms(tab, len(ws), C.c_float(mu), k, bh, block[1], None)
    nu = np.empty(S, np.float64)
    lib().orc_structure_norms(tab, len(ws), C.c_float(mu), k, bh, block[1], _ptr(nu))
    return nu


def cstep_prune(ws, lams, s: float, mu: float, fuse: Sequence[str] = ()) -> Outputs:
    tab, out, keep = _table(ws, lams)
    r = _Result()
    rc = lib().orc_cstep_prune(tab, len(ws), float(s), C.c_float(mu), fuse_bits(fuse), C.byref(r))
    assert rc == 0
    out.result = _result(r)
    return out


def cstep_filter(ws, lams, s: float, mu: float, fuse: Sequence[str] = ()) -> Outputs:
    tab, out, keep = _table(ws, lams)
    r = _Result()
    rc = lib().orc_cstep_filter(tab, len(ws), float(s), C.c_float(mu), fuse_bits(fuse), C.byref(r))
    assert rc == 0
    out.result = _result(r)
    return out


def cstep_structure(ws, lams, s: float, mu: float, kinds: Sequence[str] = ("filter", "neuron"),
                    fuse: Sequence[str] = ()) -> Outputs:
    """Rank leading-index slices: 'filter' (4-D tensors) and/or 'neuron' (rows of 2-D tensors)."""
    tab, out, keep = _table(ws, lams)
    r = _Result()
    mask = sum({"filter": 1, "neuron": 2}[k] for k in set(kinds))
    rc = lib().orc_cstep_structure(tab, len(ws), float(s), C.c_float(mu), mask, fuse_bits(fuse), C.byref(r))
    assert rc == 0
    out.result = _result(r)
    return out


def cstep_block(ws, lams, s: float, mu: float, block=(4, 4), fuse: Sequence[str] = ()) -> Outputs:
    tab, out, keep = _table(ws, lams)
    r = _Result()
    rc = lib().orc_cstep_block(tab, len(ws), float(s), C.c_float(mu), int(block[0]), int(block[1]),
                               fuse_bits(fuse), C.byref(r))
    assert rc == 0
    out.result = _result(r)
    return out


def cstep_quantize(ws, lams, mu: float, fuse: Sequence[str] = ()) -> Outputs:
    tab, out, keep = _table(ws, lams)
    rc = lib().orc_cstep_quantize(tab, len(ws), C.c_float(mu), fuse_bits(fuse))
    assert rc == 0
    return out


def lagrange_update(ws, thetas, lams, mu: float, fuse: Sequence[str] = ("lambda",)) -> Outputs:
    tab, out, keep = _table(ws, lams, thetas)
    rc = lib().orc_lagrange_update(tab, len(ws), C.c_float(mu), fuse_bits(fuse))
    assert rc == 0
    return out


def run_config(ws) -> Outputs:
    """Run the call a ``workloads.WeightSet`` names (duck typed: only its fields are read)."""
    if ws.op == "prune":
        return cstep_prune(ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse)
    if ws.op == "filter":
        return cstep_filter(ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse)
    if ws.op == "block":
        return cstep_block(ws.w, ws.lam, ws.sparsity, ws.mu, ws.block, ws.fuse)
    raise ValueError(ws.op)


def lstep_update(ws, thetas, lams, grads, buf1, buf2, mu: float, kind: str = "sgd", lr: float = 0.1,
                 momentum: float = 0.9, weight_decay: float = 0.0, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, step: int = 1):
    """One optimizer step with the penalty gradient folded in. Returns new (w, buf1, buf2) lists;
    the inputs are left untouched. ``buf1``/``buf2`` entries may be None where unused."""
    T = len(ws)
    tab = (_OptTensor * max(T, 1))()
    keep, w_out, b1_out, b2_out = [], [], [], []
    for t in range(T):
        w = np.ascontiguousarray(ws[t], dtype=np.float32).copy()
        th = np.ascontiguousarray(thetas[t], dtype=np.float32)
        lam = None if lams is None or lams[t] is None else np.ascontiguousarray(lams[t], dtype=np.float32)
        g = np.ascontiguousarray(grads[t], dtype=np.float32)
        b1 = None if buf1 is None or buf1[t] is None else np.ascontiguousarray(buf1[t], dtype=np.float32).copy()
        b2 = None if buf2 is None or buf2[t] is None else np.ascontiguousarray(buf2[t], dtype=np.float32).copy()
        keep += [th, lam, g]
        e = tab[t]
        e.w, e.theta, e.lam, e.grad, e.buf1, e.buf2 = _ptr(w), _ptr(th), _ptr(lam), _ptr(g), _ptr(b1), _ptr(b2)
        e.numel = w.size
        w_out.append(w); b1_out.append(b1); b2_out.append(b2)
    o = _Opt({"sgd": 0, "adam": 1}[kind], lr, momentum, weight_decay, beta1, beta2, eps, step)
    rc = lib().orc_lstep_update(tab, T, C.c_float(mu), C.byref(o))
    assert rc == 0
    return w_out, b1_out, b2_out


# ---------------------------------------------------------------- thinning
# Paper, Implementation ("Network Thinning"): zero structures are found and
# removed. Evaluation, Objective 1: the footprint counts non-zero parameters.
def thin_flags(theta3: np.ndarray, axis: int) -> np.ndarray:
    """theta3: array of shape [d0, d1, inner]. keep[i] = 1 iff slice i along
    ``axis`` (0 or 1) holds a value that is not zero (+0 and -0 are zero)."""
    x = np.asarray(theta3)
    assert x.ndim == 3 and axis in (0, 1)
    d = x.shape[axis]
    keep = np.zeros(d, dtype=np.uint8)
    for i in range(d):
        sl = x[i, :, :] if axis == 0 else x[:, i, :]
        keep[i] = 1 if np.any(sl != 0) else 0
    return keep


def thin_compact(src3: np.ndarray, keep0: Optional[np.ndarray], keep1: Optional[np.ndarray]) -> np.ndarray:
    """The dense tensor of the entries src3[i, j, :] whose flags keep0[i] and
    keep1[j] are non-zero, original order kept (None keeps the whole axis)."""
    x = np.asarray(src3)
    rows = [i for i in range(x.shape[0]) if keep0 is None or keep0[i] != 0]
    cols = [j for j in range(x.shape[1]) if keep1 is None or keep1[j] != 0]
    out = np.empty((len(rows), len(cols), x.shape[2]), dtype=x.dtype)
    for a, i in enumerate(rows):
        for b, j in enumerate(cols):
            out[a, b, :] = x[i, j, :]
    return out


def count_nonzero(arrays) -> np.ndarray:
    """Non-zero values per array, then their total (length T + 1, int64)."""
    c = [int(np.sum(np.asarray(a).reshape(-1) != 0)) for a in arrays]
    return np.array(c + [sum(c)], dtype=np.int64)


def footprint_bytes(arrays, bytes_per_value: int) -> int:
    """Bytes taken by the non-zero parameters (Objective 1)."""
    return int(count_nonzero(arrays)[-1]) * int(bytes_per_value)
