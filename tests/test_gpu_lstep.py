"""The fused L-step update (penalty gradient + SGD-momentum / Adam step) against the
oracle: same single fp32 operations in the same order, so every bit must agree."""
import numpy as np
import pytest

import oracle
from paper_1911_02497_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _dev(arrs, off):
    import torch
    out, keep = [], []
    for a in arrs:
        if a is None:
            out.append(None)
            continue
        buf = torch.zeros(a.size + off + 16, dtype=torch.float32, device="cuda:0")
        v = buf[off:off + a.size]
        v.copy_(torch.from_numpy(np.ascontiguousarray(a, np.float32).reshape(-1)))
        keep.append(buf)
        out.append(v)
    return out, keep


@pytest.mark.parametrize("kind", ["sgd", "adam"])
@pytest.mark.parametrize("off", [0, 3])
def test_lstep_matches_oracle(kind, off):
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    shapes = [(70001,), (33, 17), (5, 3, 3, 3), (1,), (4096,), (12289,)]
    ws = W.random_set(shapes, seed=31, kind="normal", scale=0.5, lam_sigma=1e-2, mu=1e-2)
    w = [a.reshape(-1) for a in ws.w]
    th = [np.where(np.abs(a) > 0.4, a, 0).astype(np.float32) for a in w]
    lam = [a.reshape(-1) for a in ws.lam]
    lam[2] = None                                           # a tensor without multipliers
    g = [W.draw(a.size, "normal", 1.0, 32, 0, i) for i, a in enumerate(w)]
    b1 = [W.draw(a.size, "normal", 0.1, 33, 0, i) for i, a in enumerate(w)]
    b2 = [np.abs(W.draw(a.size, "normal", 0.1, 34, 0, i)) for i, a in enumerate(w)] if kind == "adam" else None
    kw = dict(lr=0.05, momentum=0.9, weight_decay=1e-4) if kind == "sgd" else dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=5)
    for rounds in range(2):                                 # two consecutive steps
        ew, eb1, eb2 = oracle.lstep_update(w, th, lam, g, b1, b2, ws.mu, kind, **kw)
        allv, keep = _dev(w + th + g + b1 + (b2 or []) + [l for l in lam], off)
        n = len(w)
        dw, dth, dg, db1 = allv[0:n], allv[n:2 * n], allv[2 * n:3 * n], allv[3 * n:4 * n]
        db2 = allv[4 * n:5 * n] if b2 else None
        dl = allv[(5 if b2 else 4) * n:]
        tab = cstep.opt_table(dw, dth, dl, dg, db1, db2)
        ctx.lstep_update(tab, n, ws.mu, kind=kind, **kw)
        torch.cuda.synchronize()
        for t in range(n):
            assert np.array_equal(dw[t].cpu().numpy().view(np.uint32), ew[t].view(np.uint32)), (kind, t)
            assert np.array_equal(db1[t].cpu().numpy().view(np.uint32), eb1[t].view(np.uint32)), (kind, t)
            if b2:
                assert np.array_equal(db2[t].cpu().numpy().view(np.uint32), eb2[t].view(np.uint32)), (kind, t)
        w, b1, b2 = ew, eb1, (eb2 if b2 else None)
        if kind == "adam":
            kw["step"] += 1
    ctx.close()


def test_lstep_plain_sgd_without_momentum_and_argument_errors():
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    w = W.draw(5000, "normal", 1.0, 1, 0, 0); th = np.zeros_like(w); g = W.draw(5000, "normal", 1.0, 2, 0, 0)
    ew, _, _ = oracle.lstep_update([w], [th], [None], [g], None, None, 0.5, "sgd", lr=0.1, momentum=0.0)
    (dw, dth, dg), keep = _dev([w, th, g], 0)
    ctx.lstep_update(cstep.opt_table([dw], [dth], None, [dg]), 1, 0.5, kind="sgd", lr=0.1, momentum=0.0)
    torch.cuda.synchronize()
    assert np.array_equal(dw.cpu().numpy().view(np.uint32), ew[0].view(np.uint32))
    with pytest.raises(cstep.CondensaError):            # momentum without a buffer
        ctx.lstep_update(cstep.opt_table([dw], [dth], None, [dg]), 1, 0.5, kind="sgd", lr=0.1, momentum=0.9)
    with pytest.raises(cstep.CondensaError):            # theta on top of w
        ctx.lstep_update(cstep.opt_table([dw], [dw], None, [dg]), 1, 0.5, kind="sgd", lr=0.1, momentum=0.0)
    with pytest.raises(cstep.CondensaError):            # Adam without its moments
        ctx.lstep_update(cstep.opt_table([dw], [dth], None, [dg]), 1, 0.5, kind="adam")
    ctx.close()
