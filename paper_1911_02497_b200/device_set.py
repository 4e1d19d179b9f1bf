"""Device-resident copy of a weight set plus the call into the C ABI.

PyTorch is used for device memory and streams only; all arithmetic happens in
``libcondensa_cstep.so``. Used by the GPU tests, ``bench.py`` and the smoke run.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import cstep


class DeviceSet:
    """w / lambda / theta / mask / grad / theta_h buffers of a tensor list on one GPU.

    ``elem_offset`` shifts every buffer by that many elements from a 256-byte
    aligned base (to exercise the unaligned paths); ``skew`` gives theta a
    different shift so that the arrays of one tensor disagree in alignment.
    """

    def __init__(self, w: Sequence[np.ndarray], lam: Optional[Sequence[Optional[np.ndarray]]],
                 device: str = "cuda:0", with_mask=True, with_grad=True, with_theta_h=True,
                 elem_offset: int = 0, skew: int = 0, theta: Optional[Sequence[np.ndarray]] = None):
        self.device = torch.device(device)
        self.shapes = [tuple(a.shape) for a in w]
        self.T = len(w)
        self.off, self.skew = elem_offset, skew
        self._base = []            # keeps the padded allocations alive

        def alloc(n, dtype, shift):
            # guard bands: `shift` elements before and 64 behind the data carry a canary that
            # fetch() checks - a kernel that writes outside its tensor is caught here
            buf = torch.zeros(n + shift + 64, dtype=dtype, device=self.device)
            canary = self._canary(dtype)
            buf[:shift] = canary
            buf[shift + n:] = canary
            self._base.append((buf, shift, n, canary))
            return buf[shift:shift + n]

        def put(a, shift):
            t = alloc(a.size, torch.float32, shift)
            t.copy_(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32).reshape(-1)))
            return t

        self.w = [put(a, elem_offset) for a in w]
        self.lam_init = [None if (lam is None or l is None) else np.ascontiguousarray(l, np.float32)
                         for l in (lam if lam is not None else [None] * self.T)]
        self.lam = [None if l is None else put(l, elem_offset) for l in self.lam_init]
        sizes = [int(np.prod(s)) for s in self.shapes]
        if theta is None:
            self.theta = [alloc(n, torch.float32, elem_offset + skew) for n in sizes]
        else:
            self.theta = [put(a, elem_offset + skew) for a in theta]
        self.mask = [alloc(n, torch.uint8, elem_offset) for n in sizes] if with_mask else None
        self.grad = [alloc(n, torch.float32, elem_offset) for n in sizes] if with_grad else None
        self.theta_h = [alloc(n, torch.int16, elem_offset) for n in sizes] if with_theta_h else None
        lam_ptrs = [None if l is None else l for l in self.lam]
        self.table = cstep.tensor_table(self.w, lam_ptrs, self.theta, self.mask, self.grad,
                                        self.theta_h, shapes=self.shapes)

    @staticmethod
    def _canary(dtype):
        return {torch.float32: -12345.678, torch.uint8: 0xA5, torch.int16: 0x5A5A}[dtype]

    def check_guard_bands(self):
        """Raises if anything has been written next to a buffer."""
        for i, (buf, shift, n, canary) in enumerate(self._base):
            want = torch.tensor(canary, dtype=buf.dtype, device=buf.device)
            if not (bool((buf[:shift] == want).all()) and bool((buf[shift + n:] == want).all())):
                raise AssertionError("guard band of buffer %d (%s, %d elements) was overwritten" % (i, buf.dtype, n))

    # -- state ---------------------------------------------------------------
    def reset_lambda(self):
        """Restore the multipliers (they are updated in place by the calls)."""
        if getattr(self, "_lam_pristine", None) is None:
            self._lam_pristine = [None if t is None else torch.from_numpy(l.reshape(-1)).to(self.device)
                                  for t, l in zip(self.lam, self.lam_init)]
        for t, p in zip(self.lam, self._lam_pristine):
            if t is not None:
                t.copy_(p)

    def poison_outputs(self):
        """Fill every output with a recognisable pattern so that skipped writes show."""
        for t in self.theta:
            t.fill_(float("nan"))
        for group, val in ((self.mask, 7), (self.grad, float("nan")), (self.theta_h, 0x5555)):
            if group is not None:
                for t in group:
                    t.fill_(val)

    # -- calls ---------------------------------------------------------------
    def run(self, ctx: "cstep.Context", op: str, sparsity: float = 0.0, mu: float = 1e-3,
            fuse=(), block=(4, 4), stream=None):
        if op == "prune":
            ctx.cstep_prune(self.table, self.T, sparsity, mu, fuse, stream)
        elif op == "filter":
            ctx.cstep_filter(self.table, self.T, sparsity, mu, fuse, stream)
        elif op in ("neuron", "structure"):
            kinds = ("neuron",) if op == "neuron" else ("filter", "neuron")
            ctx.cstep_structure(self.table, self.T, sparsity, mu, kinds, fuse, stream)
        elif op == "block":
            ctx.cstep_block(self.table, self.T, sparsity, mu, block[0], block[1], fuse, stream)
        elif op.startswith("quantize"):
            dt = {"quantize": cstep.DTYPE_FP16, "quantize_bf16": cstep.DTYPE_BF16,
                  "quantize_e4m3": cstep.DTYPE_FP8_E4M3, "quantize_e5m2": cstep.DTYPE_FP8_E5M2}[op]
            ctx.cstep_quantize(self.table, self.T, mu, dt, fuse, stream)
        elif op == "lagrange":
            ctx.cstep_lagrange_update(self.table, self.T, mu, fuse, stream)
        else:
            raise ValueError(op)

    # -- read back -----------------------------------------------------------
    def _get(self, group, dtype) -> Optional[List[np.ndarray]]:
        if group is None:
            return None
        return [None if t is None else t.cpu().numpy().view(dtype).reshape(s)
                for t, s in zip(group, self.shapes)]

    def fetch(self):
        torch.cuda.synchronize(self.device)
        self.check_guard_bands()
        return {"theta": self._get(self.theta, np.float32), "mask": self._get(self.mask, np.uint8),
                "lam": self._get(self.lam, np.float32), "grad": self._get(self.grad, np.float32),
                "theta_h": self._get(self.theta_h, np.uint16)}

    @property
    def numel(self) -> int:
        return int(sum(int(np.prod(s)) for s in self.shapes))
