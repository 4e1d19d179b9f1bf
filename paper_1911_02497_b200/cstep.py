"""Thin ctypes binding of ``libcondensa_cstep.so`` (argument marshalling only).

Every step of the C-step runs in the library's CUDA kernels; PyTorch is used
by callers for device memory and streams. There is no CPU fallback: if the
shared library is missing or no CUDA device is present the calls raise.
Function names and arguments mirror ``include/condensa_cstep.h``.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcondensa_cstep.so")

FUSE_FP16, FUSE_LAMBDA, FUSE_PENALTY, NO_SAMPLING = 1, 2, 4, 64
OP_PRUNE, OP_FILTER, OP_BLOCK, OP_QUANTIZE, OP_LAGRANGE = 0, 1, 2, 3, 4
DTYPE_FP16, DTYPE_BF16, DTYPE_FP8_E4M3, DTYPE_FP8_E5M2 = 1, 2, 3, 4
FUSE_BF16, FUSE_E4M3, FUSE_E5M2 = 8, 16, 32
STRUCT_FILTER, STRUCT_NEURON = 1, 2
OK, ERR_INVALID_ARG, ERR_WORKSPACE, ERR_CUDA, ERR_UNSUPPORTED, ERR_INTERNAL = 0, -1, -2, -3, -4, -5
ERR_TOO_LARGE = -6
NOALLOC_MAX_NUMEL = 1048576

EXPORTS = ["condensa_create", "condensa_destroy", "condensa_cstep_prune", "condensa_cstep_filter",
           "condensa_cstep_block", "condensa_cstep_quantize", "condensa_cstep_lagrange_update",
           "condensa_cstep_host", "condensa_get_result", "condensa_launch_count",
           "condensa_last_error", "condensa_profile_enable", "condensa_profile_read",
           "condensa_cstep_prune_noalloc", "condensa_lstep_update",
           "condensa_cstep_structure", "condensa_thin_flags", "condensa_thin_compact",
           "condensa_count_nonzero", "condensa_set_seed", "condensa_noalloc_status",
           "condensa_cstep_structured", "condensa_workspace_bytes", "condensa_thin_list"]


class CondensaError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("condensa error %d: %s" % (code, text))
        self.code = code


class Tensor(C.Structure):
    """Mirror of ``condensa_tensor``."""
    _fields_ = [("w", C.c_void_p), ("lam", C.c_void_p), ("theta", C.c_void_p),
                ("mask", C.c_void_p), ("grad", C.c_void_p), ("theta_h", C.c_void_p),
                ("numel", C.c_int64), ("ndim", C.c_int32), ("shape", C.c_int64 * 4)]


class Result(C.Structure):
    """Mirror of ``condensa_result``."""
    _fields_ = [("status", C.c_int32), ("passes", C.c_int32), ("n_units", C.c_int64),
                ("n_zero", C.c_int64), ("n_keep", C.c_int64), ("tau_key", C.c_uint64),
                ("tau_id", C.c_int64), ("n_gt", C.c_int64), ("n_tie", C.c_int64),
                ("n_tie_kept", C.c_int64), ("tau_norm", C.c_float), ("sampled", C.c_int32),
                ("n_candidates", C.c_int64), ("n_repaired", C.c_int64), ("seed", C.c_uint64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class StructureSpec(C.Structure):
    """Mirror of ``condensa_structure_spec``."""
    _fields_ = [("kind", C.c_int32), ("kinds", C.c_int32), ("criterion", C.c_int32), ("ndim", C.c_int32),
                ("block", C.c_int64 * 4)]


SPEC_SLICES, SPEC_BLOCKS = 0, 1
CRITERIA = {"l2": 0, "l1": 1, "max": 2}


class ThinLayer(C.Structure):
    """Mirror of ``condensa_thin_layer``."""
    _fields_ = [("src", C.c_void_p), ("d0", C.c_int64), ("d1", C.c_int64), ("inner", C.c_int64),
                ("keep0", C.c_void_p), ("remove_axis0", C.c_int32), ("keep1_from", C.c_int32),
                ("dst", C.c_void_p), ("dims_out", C.c_void_p)]


class OptTensor(C.Structure):
    """Mirror of ``condensa_opt_tensor``."""
    _fields_ = [("w", C.c_void_p), ("theta", C.c_void_p), ("lam", C.c_void_p), ("grad", C.c_void_p),
                ("buf1", C.c_void_p), ("buf2", C.c_void_p), ("numel", C.c_int64)]


class Opt(C.Structure):
    """Mirror of ``condensa_opt``."""
    _fields_ = [("kind", C.c_int32), ("lr", C.c_float), ("momentum", C.c_float),
                ("weight_decay", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("step", C.c_int64)]


OPT_SGD, OPT_ADAM = 0, 1


class KernelTime(C.Structure):
    """Mirror of ``condensa_kernel_time``."""
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int64), ("total_ms", C.c_double)]


_lib = None


def load():
    """Load the shared library (no GPU needed for this) and declare signatures."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: run `python -m paper_1911_02497_b200.build`" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i32, u32, f32, f64 = C.c_void_p, C.c_int, C.c_uint, C.c_float, C.c_double
    L.condensa_create.argtypes = [C.POINTER(vp), i32, C.c_size_t]
    L.condensa_destroy.argtypes = [vp]
    L.condensa_cstep_prune.argtypes = [vp, vp, i32, f64, f32, u32, vp]
    L.condensa_cstep_filter.argtypes = [vp, vp, i32, f64, f32, u32, vp]
    L.condensa_cstep_block.argtypes = [vp, vp, i32, f64, f32, i32, i32, u32, vp]
    L.condensa_cstep_structure.argtypes = [vp, vp, i32, f64, f32, i32, u32, vp]
    L.condensa_cstep_quantize.argtypes = [vp, vp, i32, f32, i32, u32, vp]
    L.condensa_cstep_structured.argtypes = [vp, vp, i32, f64, f32, C.POINTER(StructureSpec), u32, vp]
    L.condensa_cstep_lagrange_update.argtypes = [vp, vp, i32, f32, u32, vp]
    L.condensa_cstep_host.argtypes = [vp, i32, vp, i32, f64, f32, i32, i32, u32, vp]
    L.condensa_get_result.argtypes = [vp, C.POINTER(Result)]
    L.condensa_profile_enable.argtypes = [vp, i32]
    L.condensa_profile_read.argtypes = [vp, C.POINTER(KernelTime), i32, C.POINTER(i32)]
    L.condensa_cstep_prune_noalloc.argtypes = [vp, f64, f32, u32, vp]
    L.condensa_noalloc_status.argtypes = []
    L.condensa_workspace_bytes.argtypes = [i32, vp, i32, C.POINTER(StructureSpec), u32, C.POINTER(C.c_size_t)]
    L.condensa_set_seed.argtypes = [vp, C.c_uint64]
    L.condensa_lstep_update.argtypes = [vp, vp, i32, f32, C.POINTER(Opt), vp]
    i64 = C.c_int64
    L.condensa_thin_flags.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp]
    L.condensa_thin_compact.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp, vp]
    L.condensa_count_nonzero.argtypes = [vp, C.POINTER(vp), C.POINTER(i64), i32, vp, vp]
    L.condensa_thin_list.argtypes = [vp, C.POINTER(ThinLayer), i32, vp]
    L.condensa_launch_count.argtypes = [vp]
    L.condensa_launch_count.restype = C.c_int64
    L.condensa_last_error.argtypes = [vp]
    L.condensa_last_error.restype = C.c_char_p
    for name in EXPORTS:
        getattr(L, name)
    _lib = L
    return L


def fuse_bits(fuse) -> int:
    if isinstance(fuse, int):
        return fuse
    table = {"fp16": FUSE_FP16, "lambda": FUSE_LAMBDA, "penalty": FUSE_PENALTY, "bf16": FUSE_BF16,
             "e4m3": FUSE_E4M3, "e5m2": FUSE_E5M2, "no_sampling": NO_SAMPLING}
    b = 0
    for f in fuse:
        b |= table[f]
    return b


def _addr(x) -> Optional[int]:
    """Address of a torch tensor, a numpy array, an int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    return int(x.ctypes.data)


def tensor_table(w: Sequence, lam: Optional[Sequence] = None, theta: Optional[Sequence] = None,
                 mask: Optional[Sequence] = None, grad: Optional[Sequence] = None,
                 theta_h: Optional[Sequence] = None, shapes: Optional[Sequence] = None):
    """Build a ``condensa_tensor[T]`` array from per-tensor buffers (torch tensors
    on the device, or numpy arrays for the host entry point). Buffers must be
    contiguous; the caller keeps them alive."""
    T = len(w)
    tab = (Tensor * max(T, 1))()
    for t in range(T):
        e = tab[t]
        shp = tuple(shapes[t]) if shapes is not None else tuple(w[t].shape)
        n = 1
        for d in shp:
            n *= int(d)
        e.w = _addr(w[t])
        e.lam = _addr(lam[t]) if lam is not None else None
        e.theta = _addr(theta[t]) if theta is not None else None
        e.mask = _addr(mask[t]) if mask is not None else None
        e.grad = _addr(grad[t]) if grad is not None else None
        e.theta_h = _addr(theta_h[t]) if theta_h is not None else None
        e.numel, e.ndim = n, len(shp)
        for d in range(4):
            e.shape[d] = int(shp[d]) if d < len(shp) else 1
    return tab


def opt_table(w, theta, lam, grad, buf1=None, buf2=None):
    """``condensa_opt_tensor[T]`` from per-tensor device buffers (entries of lam/buf1/buf2 may be None)."""
    T = len(w)
    tab = (OptTensor * max(T, 1))()
    for t in range(T):
        e = tab[t]
        e.w, e.theta, e.grad = _addr(w[t]), _addr(theta[t]), _addr(grad[t])
        e.lam = _addr(lam[t]) if lam is not None else None
        e.buf1 = _addr(buf1[t]) if buf1 is not None else None
        e.buf2 = _addr(buf2[t]) if buf2 is not None else None
        e.numel = int(w[t].numel()) if hasattr(w[t], "numel") else int(w[t].size)
    return tab


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)          # torch.cuda.Stream


def cstep_prune_noalloc(tab, sparsity, mu, fuse=(), stream=None):
    """``condensa_cstep_prune_noalloc``: magnitude pruning of ONE tensor (entry 0 of
    ``tab``) on the current CUDA device without any device allocation by the
    library - for callers whose memory pool owns the whole device or who cannot
    take cudaMalloc's synchronisation. At most ``NOALLOC_MAX_NUMEL`` elements;
    calls on one device must not overlap (they share one built-in scratch)."""
    L = load()
    rc = L.condensa_cstep_prune_noalloc(tab, float(sparsity), float(mu), fuse_bits(fuse),
                                        _stream_handle(stream))
    if rc != OK:
        raise CondensaError(rc, (L.condensa_last_error(None) or b"").decode())


def workspace_bytes(op: int, tab, T: int, fuse=(), spec=None) -> int:
    """``condensa_workspace_bytes``: what ``Context(device, workspace_bytes)`` must reserve so that
    calls of this shape never allocate."""
    L = load()
    n = C.c_size_t(0)
    rc = L.condensa_workspace_bytes(int(op), tab, int(T), spec, fuse_bits(fuse), C.byref(n))
    if rc != OK:
        raise CondensaError(rc, (L.condensa_last_error(None) or b"").decode())
    return int(n.value)


def noalloc_status():
    """``condensa_noalloc_status``: waits for the last allocation-free call on the current
    device and raises if one of its device-side checks failed."""
    L = load()
    rc = L.condensa_noalloc_status()
    if rc != OK:
        raise CondensaError(rc, (L.condensa_last_error(None) or b"").decode())


class Context:
    """Owns a ``condensa_ctx`` (workspace and descriptor cache of one device)."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._lib = load()
        h = C.c_void_p()
        rc = self._lib.condensa_create(C.byref(h), int(device), int(workspace_bytes))
        if rc != OK:
            raise CondensaError(rc, (self._lib.condensa_last_error(None) or b"").decode())
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.condensa_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise CondensaError(rc, (self._lib.condensa_last_error(self._h) or b"").decode())

    def set_seed(self, seed: int):
        self._check(self._lib.condensa_set_seed(self._h, int(seed) & ((1 << 64) - 1)))

    def cstep_prune(self, tab, T, sparsity, mu, fuse=(), stream=None):
        self._check(self._lib.condensa_cstep_prune(self._h, tab, T, float(sparsity), float(mu),
                                                   fuse_bits(fuse), _stream_handle(stream)))

    def cstep_filter(self, tab, T, sparsity, mu, fuse=(), stream=None):
        self._check(self._lib.condensa_cstep_filter(self._h, tab, T, float(sparsity), float(mu),
                                                    fuse_bits(fuse), _stream_handle(stream)))

    def cstep_structure(self, tab, T, sparsity, mu, kinds=("filter", "neuron"), fuse=(), stream=None):
        mask = sum({"filter": STRUCT_FILTER, "neuron": STRUCT_NEURON}[k] for k in set(kinds))
        self._check(self._lib.condensa_cstep_structure(self._h, tab, T, float(sparsity), float(mu), mask,
                                                       fuse_bits(fuse), _stream_handle(stream)))

    def cstep_structured(self, tab, T, sparsity, mu, kind="filter", block=None, criterion="l2", fuse=(), stream=None):
        """``kind``: 'filter', 'neuron', 'structure' (both) or 'block' with ``block`` = the extents."""
        sp = StructureSpec()
        sp.criterion = CRITERIA[criterion]
        if kind == "block":
            sp.kind, sp.ndim = SPEC_BLOCKS, len(block)
            for d, b in enumerate(block):
                sp.block[d] = int(b)
        else:
            sp.kind, sp.kinds = SPEC_SLICES, {"filter": 1, "neuron": 2, "structure": 3}[kind]
        self._check(self._lib.condensa_cstep_structured(self._h, tab, T, float(sparsity), float(mu), C.byref(sp),
                                                        fuse_bits(fuse), _stream_handle(stream)))

    def cstep_block(self, tab, T, sparsity, mu, bh=4, bw=4, fuse=(), stream=None):
        self._check(self._lib.condensa_cstep_block(self._h, tab, T, float(sparsity), float(mu),
                                                   int(bh), int(bw), fuse_bits(fuse),
                                                   _stream_handle(stream)))

    def cstep_quantize(self, tab, T, mu, dtype=DTYPE_FP16, fuse=(), stream=None):
        self._check(self._lib.condensa_cstep_quantize(self._h, tab, T, float(mu), int(dtype),
                                                      fuse_bits(fuse), _stream_handle(stream)))

    def cstep_lagrange_update(self, tab, T, mu, fuse=("lambda",), stream=None):
        self._check(self._lib.condensa_cstep_lagrange_update(self._h, tab, T, float(mu),
                                                             fuse_bits(fuse), _stream_handle(stream)))

    def cstep_host(self, op, tab, T, sparsity, mu, bh=4, bw=4, fuse=(), stream=None):
        self._check(self._lib.condensa_cstep_host(self._h, int(op), tab, T, float(sparsity),
                                                  float(mu), int(bh), int(bw), fuse_bits(fuse),
                                                  _stream_handle(stream)))

    def lstep_update(self, tab, T, mu, kind="sgd", lr=0.1, momentum=0.9, weight_decay=0.0, beta1=0.9,
                     beta2=0.999, eps=1e-8, step=1, stream=None):
        o = Opt({"sgd": OPT_SGD, "adam": OPT_ADAM}[kind], lr, momentum, weight_decay, beta1, beta2, eps, step)
        self._check(self._lib.condensa_lstep_update(self._h, tab, T, float(mu), C.byref(o),
                                                    _stream_handle(stream)))

    def thin_flags(self, theta, d0, d1, inner, axis, keep, stream=None):
        self._check(self._lib.condensa_thin_flags(self._h, _addr(theta), int(d0), int(d1), int(inner), int(axis),
                                                  _addr(keep), _stream_handle(stream)))

    def thin_compact(self, src, d0, d1, inner, keep0, keep1, dst, dims_out, stream=None):
        self._check(self._lib.condensa_thin_compact(self._h, _addr(src), int(d0), int(d1), int(inner),
                                                    _addr(keep0), _addr(keep1), _addr(dst), _addr(dims_out),
                                                    _stream_handle(stream)))

    def thin_list(self, layers, stream=None):
        """``layers``: dicts with src, d0, d1, inner, keep0, remove_axis0, keep1_from, dst, dims_out."""
        n = len(layers)
        tab = (ThinLayer * max(n, 1))()
        for e, x in zip(tab, layers):
            e.src, e.dst, e.keep0, e.dims_out = _addr(x["src"]), _addr(x["dst"]), _addr(x["keep0"]), _addr(x["dims_out"])
            e.d0, e.d1, e.inner = int(x["d0"]), int(x["d1"]), int(x["inner"])
            e.remove_axis0, e.keep1_from = int(bool(x.get("remove_axis0", True))), int(x.get("keep1_from", -1))
        self._check(self._lib.condensa_thin_list(self._h, tab, n, _stream_handle(stream)))

    def count_nonzero(self, arrays, counts, stream=None):
        """``arrays``: device float32 tensors; ``counts``: device int64 tensor of len(arrays) + 1."""
        T = len(arrays)
        ptrs = (C.c_void_p * max(T, 1))(*[_addr(a) for a in arrays])
        numel = (C.c_int64 * max(T, 1))(*[int(a.numel()) for a in arrays])
        self._check(self._lib.condensa_count_nonzero(self._h, ptrs, numel, T, _addr(counts),
                                                     _stream_handle(stream)))

    def get_result(self) -> Result:
        r = Result()
        self._check(self._lib.condensa_get_result(self._h, C.byref(r)))
        return r

    def profile_enable(self, on: bool):
        self._check(self._lib.condensa_profile_enable(self._h, 1 if on else 0))

    def profile_read(self):
        """{kernel name: (launches, total ms)} since profiling was enabled."""
        buf = (KernelTime * 32)()
        n = C.c_int(0)
        self._check(self._lib.condensa_profile_read(self._h, buf, 32, C.byref(n)))
        return {buf[i].name.decode(): (int(buf[i].launches), float(buf[i].total_ms))
                for i in range(n.value)}

    def launch_count(self) -> int:
        return int(self._lib.condensa_launch_count(self._h))
