"""Thinning kernels (zero-structure flags, compaction, non-zero count) against the
oracle: byte and bit exact. Paper, Implementation ("Network Thinning")."""
import numpy as np
import pytest

import oracle
from paper_1911_02497_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _dev(a, off=0):
    import torch
    flat = np.ascontiguousarray(a, np.float32).reshape(-1)
    buf = torch.zeros(flat.size + off + 16, dtype=torch.float32, device="cuda:0")
    v = buf[off:off + flat.size]
    v.copy_(torch.from_numpy(flat))
    return v, buf


def _structured_zeros(shape, seed, p0=0.35, p1=0.3, sprinkle=0.5):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(shape).astype(np.float32)
    x[rng.random(shape) < sprinkle] = 0.0
    if shape[0]:
        x[rng.random(shape[0]) < p0] = 0.0
    if shape[1]:
        x[:, rng.random(shape[1]) < p1] = 0.0
    return x


def _run_compact(ctx, x3, k0, k1, off):
    import torch
    d0, d1, inner = x3.shape
    src, _b = _dev(x3, off)
    dst = torch.full((x3.size + off + 16,), float("nan"), dtype=torch.float32, device="cuda:0")[off:]
    dims = torch.full((2,), -1, dtype=torch.int64, device="cuda:0")
    dk0 = torch.from_numpy(k0).cuda() if k0 is not None else None
    dk1 = torch.from_numpy(k1).cuda() if k1 is not None else None
    ctx.thin_compact(src, d0, d1, inner, dk0, dk1, dst, dims)
    torch.cuda.synchronize()
    n0, n1 = (int(v) for v in dims.cpu())
    out = dst[:n0 * n1 * inner].cpu().numpy().reshape(n0, n1, inner)
    rest = dst[n0 * n1 * inner:x3.size].cpu().numpy()
    assert np.all(np.isnan(rest)), "wrote past the compacted tensor"
    return out


SHAPES = [(37, 19, 9), (300, 130, 1), (5000, 1, 1), (64, 48, 25), (2100, 1500, 1), (3, 4100, 3),
          (1, 1, 1), (130, 12, 4)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("off", [0, 3])
def test_flags_and_compact_match_oracle(shape, off):
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    x = _structured_zeros(shape, seed=sum(shape) + off)
    if x.size > 10:
        x.reshape(-1)[5] = np.float32(-0.0)
    src, _b = _dev(x, off)
    flags = []
    for axis in (0, 1):
        keep = torch.full((shape[axis],), 7, dtype=torch.uint8, device="cuda:0")
        ctx.thin_flags(src, shape[0], shape[1], shape[2], axis, keep)
        torch.cuda.synchronize()
        got = keep.cpu().numpy()
        assert np.array_equal(got, oracle.thin_flags(x, axis)), (shape, axis)
        flags.append(got)
    for k0, k1 in ((flags[0], flags[1]), (flags[0], None), (None, flags[1]), (None, None)):
        got = _run_compact(ctx, x, k0, k1, off)
        exp = oracle.thin_compact(x, k0, k1)
        assert got.shape == exp.shape, (shape, got.shape, exp.shape)
        assert np.array_equal(got.view(np.uint32), exp.view(np.uint32)), shape
    ctx.close()


def test_degenerate_inputs():
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    # all zero: every flag 0, nothing kept
    x = np.zeros((17, 5, 3), np.float32)
    src, _b = _dev(x)
    keep = torch.full((17,), 7, dtype=torch.uint8, device="cuda:0")
    ctx.thin_flags(src, 17, 5, 3, 0, keep)
    assert int(keep.sum()) == 0
    out = _run_compact(ctx, x, keep.cpu().numpy(), None, 0)
    assert out.shape == (0, 5, 3)
    # empty extents are accepted
    dims = torch.full((2,), -1, dtype=torch.int64, device="cuda:0")
    ctx.thin_flags(None, 0, 5, 3, 0, None)
    ctx.thin_compact(None, 0, 5, 3, None, None, None, dims)
    torch.cuda.synchronize()
    assert dims.cpu().tolist() == [0, 5]
    # a dense tensor comes back unchanged
    y = np.random.default_rng(1).standard_normal((33, 9, 4)).astype(np.float32)
    k0 = np.ones(33, np.uint8)
    assert np.array_equal(_run_compact(ctx, y, k0, np.ones(9, np.uint8), 0), y)
    # bad arguments are refused on the host
    with pytest.raises(cstep.CondensaError):
        ctx.thin_flags(src, 17, 5, 3, 2, keep)
    with pytest.raises(cstep.CondensaError):
        ctx.thin_compact(src, 17, 5, 3, None, None, src, dims)
    ctx.close()


def test_count_nonzero_matches_oracle():
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    rng = np.random.default_rng(2)
    arrs = []
    for n in (1, 4095, 4096, 4097, 70001, 0, 123457):
        a = rng.standard_normal(n).astype(np.float32)
        a[rng.random(n) < 0.8] = 0.0
        if n > 3:
            a[1], a[2] = np.float32(-0.0), np.float32(1e-45)
        arrs.append(a)
    dev = [_dev(a, 1)[0] for a in arrs]
    counts = torch.full((len(arrs) + 1,), -5, dtype=torch.int64, device="cuda:0")
    for _ in range(2):                       # the call clears the counters itself
        ctx.count_nonzero(dev, counts)
    torch.cuda.synchronize()
    assert np.array_equal(counts.cpu().numpy(), oracle.count_nonzero(arrs))
    ctx.close()


def test_thin_vgg_after_filter_pruning_full_size():
    """Config 3 at full size: filter pruning, then the chain strategy (a layer loses
    its zero filters and the input channels its predecessor lost). Flags and
    thinned tensors equal the oracle's, computed from the oracle's own theta."""
    import torch
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ws = W.config("3")
    ctx = cstep.Context(0)
    ds = DeviceSet(ws.w, ws.lam, device="cuda:0")
    ds.run(ctx, ws.op, ws.sparsity, ws.mu, ws.fuse, ws.block)
    torch.cuda.synchronize()
    exp = oracle.run_config(ws)
    prev = None
    total_before = total_after = 0
    convs = [t for t in range(len(ws.w)) if len(ws.shapes[t]) == 4]
    for t in convs:
        Fo, Ci, kh, kw = ws.shapes[t]
        th = ds.theta[t]
        keep0 = torch.empty(Fo, dtype=torch.uint8, device="cuda:0")
        ctx.thin_flags(th, Fo, Ci, kh * kw, 0, keep0)
        e3 = exp.theta[t].reshape(Fo, Ci, kh * kw)
        ek0 = oracle.thin_flags(e3, 0)
        assert np.array_equal(keep0.cpu().numpy(), ek0), t
        dst = torch.empty(Fo * Ci * kh * kw, dtype=torch.float32, device="cuda:0")
        dims = torch.zeros(2, dtype=torch.int64, device="cuda:0")
        ctx.thin_compact(th, Fo, Ci, kh * kw, keep0, prev, dst, dims)
        torch.cuda.synchronize()
        n0, n1 = (int(v) for v in dims.cpu())
        eprev = prev.cpu().numpy() if prev is not None else None
        eout = oracle.thin_compact(e3, ek0, eprev)
        assert (n0, n1) == eout.shape[:2], t
        got = dst[:n0 * n1 * kh * kw].cpu().numpy()
        assert np.array_equal(got.view(np.uint32), eout.reshape(-1).view(np.uint32)), t
        total_before += e3.size
        total_after += eout.size
        prev = keep0
    assert total_after < 0.2 * total_before       # 80 % of the filters went, and their channels downstream
    counts = torch.zeros(len(ws.w) + 1, dtype=torch.int64, device="cuda:0")
    ctx.count_nonzero(ds.theta, counts)
    torch.cuda.synchronize()
    assert np.array_equal(counts.cpu().numpy(), oracle.count_nonzero(exp.theta))
    ctx.close()


def _list_case(shapes, chain, seed, off=0):
    """Layers for ``Context.thin_list``: ``shapes`` are (d0, d1, inner); ``chain[l]`` is the
    layer whose axis-0 flags remove layer l's axis-1 slices (-1: none)."""
    import torch
    host, layers, keep = [], [], []
    for l, shp in enumerate(shapes):
        x = _structured_zeros(shp, seed + l)
        if chain[l] >= 0:
            assert shapes[chain[l]][0] == shp[1]
        host.append(x)
        src, buf = _dev(x, off)
        n = max(x.size, 1)
        layers.append(dict(src=src if x.size else None, d0=shp[0], d1=shp[1], inner=shp[2],
                           keep0=torch.full((max(shp[0], 1),), 7, dtype=torch.uint8, device="cuda:0"),
                           remove_axis0=(l % 3 != 2), keep1_from=chain[l],
                           dst=torch.full((n + off + 16,), float("nan"), dtype=torch.float32, device="cuda:0")[off:],
                           dims_out=torch.full((2,), -1, dtype=torch.int64, device="cuda:0"), _buf=buf))
    return host, layers


def _check_list(host, layers):
    import torch
    torch.cuda.synchronize()
    flags = [oracle.thin_flags(x, 0) for x in host]
    for l, (x, lay) in enumerate(zip(host, layers)):
        d0 = x.shape[0]
        got_flags = lay["keep0"][:d0].cpu().numpy()
        assert np.array_equal(got_flags, flags[l]), l
        k0 = flags[l] if lay["remove_axis0"] else None
        k1 = flags[lay["keep1_from"]] if lay["keep1_from"] >= 0 else None
        exp = oracle.thin_compact(x, k0, k1)
        n0, n1 = (int(v) for v in lay["dims_out"].cpu())
        assert (n0, n1) == exp.shape[:2], (l, n0, n1, exp.shape)
        got = lay["dst"][:exp.size].cpu().numpy()
        assert np.array_equal(got.view(np.uint32), exp.reshape(-1).view(np.uint32)), l
        rest = lay["dst"][exp.size:max(x.size, 1)].cpu().numpy()
        assert np.all(np.isnan(rest)), (l, "wrote past the compacted tensor")


@pytest.mark.parametrize("off", [0, 1])
def test_thin_list_matches_oracle(off):
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    # a conv chain, a classifier fed by the last conv layer, a bias, ragged and empty extents
    shapes = [(37, 3, 9), (64, 37, 9), (130, 64, 25), (300, 130, 1), (300, 1, 1), (2100, 300, 1),
              (5, 0, 3), (0, 5, 3), (1, 1, 1), (3, 4100, 3), (1500, 2100, 1)]
    chain = [-1, 0, 1, 2, -1, 3, -1, -1, -1, -1, 5]
    host, layers = _list_case(shapes, chain, seed=50 + off, off=off)
    for _ in range(2):                       # a second call on the same context reuses the workspace
        ctx.thin_list(layers)
    _check_list(host, layers)
    ctx.close()


def test_thin_list_refuses_bad_arguments():
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    host, layers = _list_case([(8, 4, 2), (6, 7, 2)], [-1, -1], seed=3)
    with pytest.raises(cstep.CondensaError):
        ctx.thin_list([])
    bad = [dict(l) for l in layers]
    bad[1]["keep1_from"] = 0                  # layer 0 has 8 filters, layer 1 has 7 input channels
    with pytest.raises(cstep.CondensaError):
        ctx.thin_list(bad)
    bad = [dict(l) for l in layers]
    bad[0]["dst"] = bad[0]["src"]
    with pytest.raises(cstep.CondensaError):
        ctx.thin_list(bad)
    ctx.thin_list(layers)                     # the context is still usable
    _check_list(host, layers)
    ctx.close()


def test_thin_list_vgg_full_size_equals_per_layer_calls():
    """Config 3 after filter pruning: the chain strategy over all conv layers in one call
    equals the oracle layer by layer."""
    import torch
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ws = W.config("3")
    ctx = cstep.Context(0)
    ds = DeviceSet(ws.w, ws.lam, device="cuda:0")
    ds.run(ctx, ws.op, ws.sparsity, ws.mu, ws.fuse, ws.block)
    torch.cuda.synchronize()
    exp = oracle.run_config(ws)
    convs = [t for t in range(len(ws.w)) if len(ws.shapes[t]) == 4]
    host, layers = [], []
    for i, t in enumerate(convs):
        Fo, Ci, kh, kw = ws.shapes[t]
        host.append(exp.theta[t].reshape(Fo, Ci, kh * kw))
        layers.append(dict(src=ds.theta[t], d0=Fo, d1=Ci, inner=kh * kw,
                           keep0=torch.empty(Fo, dtype=torch.uint8, device="cuda:0"), remove_axis0=True,
                           keep1_from=i - 1,
                           dst=torch.full((Fo * Ci * kh * kw,), float("nan"), dtype=torch.float32, device="cuda:0"),
                           dims_out=torch.zeros(2, dtype=torch.int64, device="cuda:0")))
    ctx.thin_list(layers)
    _check_list(host, layers)
    ctx.close()
