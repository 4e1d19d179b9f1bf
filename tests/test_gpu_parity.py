"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs. Integer / bit results must be identical; fp32 values are
produced by the same single IEEE operations, so they are compared bit for bit as
well (and within 1e-6 relative as the stated bar)."""
import ctypes as C
import math

import numpy as np
import pytest

import oracle
from paper_1911_02497_b200 import workloads as W

pytestmark = pytest.mark.gpu

REL = 1e-6      # tolerance stated for fp32 norms and multiplier updates


SEED = 0x5EEDC0FFEE      # sample positions of the module's context (reproducible runs)


@pytest.fixture(scope="module")
def ctx():
    from paper_1911_02497_b200 import cstep
    c = cstep.Context(0)
    c.set_seed(SEED)
    yield c
    c.close()


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def same_f32(a, b):
    """Bit-identical, except that a NaN only has to be a NaN (IEEE leaves the
    payload of a generated NaN to the implementation)."""
    a = np.ascontiguousarray(a, np.float32); b = np.ascontiguousarray(b, np.float32)
    na, nb = np.isnan(a), np.isnan(b)
    return bool(np.array_equal(na, nb) and np.array_equal(bits(a)[~na], bits(b)[~nb]))


def same_f16(a, b):
    """binary16 bit patterns agree; a NaN only has to be a NaN."""
    a = np.asarray(a, np.uint16); b = np.asarray(b, np.uint16)
    na, nb = (a & 0x7FFF) > 0x7C00, (b & 0x7FFF) > 0x7C00
    return bool(np.array_equal(na, nb) and np.array_equal(a[~na], b[~nb]))


def rel_close(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    both_nan = np.isnan(a) & np.isnan(b)
    ok = np.abs(a - b) <= REL * np.maximum(np.abs(b), 1e-30)
    return bool(np.all(ok | both_nan | (a == b)))


def run_gpu(ctx, op, w, lam, s, mu, fuse, block=(4, 4), elem_offset=0, skew=0, theta=None):
    from paper_1911_02497_b200.device_set import DeviceSet
    ds = DeviceSet(w, lam, elem_offset=elem_offset, skew=skew, theta=theta)
    ds.poison_outputs() if theta is None else None
    ds.run(ctx, op, s, mu, fuse, block)
    out = ds.fetch()
    res = ctx.get_result() if op in ("prune", "filter", "block", "neuron", "structure") else None
    return out, res


def run_oracle(op, w, lam, s, mu, fuse, block=(4, 4), theta=None):
    fuse = tuple(f for f in fuse if f != "no_sampling")     # a path switch of the CUDA side only
    if op == "prune":
        return oracle.cstep_prune(w, lam, s, mu, fuse)
    if op == "filter":
        return oracle.cstep_filter(w, lam, s, mu, fuse)
    if op in ("neuron", "structure"):
        return oracle.cstep_structure(w, lam, s, mu, ("neuron",) if op == "neuron" else ("filter", "neuron"), fuse)
    if op == "block":
        return oracle.cstep_block(w, lam, s, mu, block, fuse)
    if op == "quantize":
        return oracle.cstep_quantize(w, lam, mu, fuse)
    if op.startswith("quantize_"):
        return oracle.cstep_quantize(w, lam, mu, tuple(fuse) + (op.split("_")[1],))
    return oracle.lagrange_update(w, theta, lam, mu, fuse)


def check(ctx, op, w, lam, s=0.0, mu=1e-3, fuse=("lambda",), block=(4, 4), elem_offset=0, skew=0,
          theta=None, exact_key=True):
    lam = lam if lam is not None else [None] * len(w)
    got, res = run_gpu(ctx, op, w, lam, s, mu, fuse, block, elem_offset, skew, theta)
    exp = run_oracle(op, w, lam, s, mu, fuse, block, theta)
    T = len(w)
    for t in range(T):
        if op != "lagrange":
            assert np.array_equal(got["mask"][t], exp.mask[t]), "mask, tensor %d" % t
            assert same_f32(got["theta"][t], exp.theta[t]), "theta, tensor %d" % t
            assert same_f16(got["theta_h"][t], exp.theta_h[t]), "theta_h, tensor %d" % t
        if lam[t] is not None:
            assert rel_close(got["lam"][t], exp.lam[t])
            assert same_f32(got["lam"][t], exp.lam[t]), "lambda, tensor %d" % t
        if "penalty" in fuse:
            assert rel_close(got["grad"][t], exp.grad[t])
            assert same_f32(got["grad"][t], exp.grad[t]), "grad, tensor %d" % t
    if res is not None:
        r = exp.result
        assert res.status == 0
        assert (res.n_units, res.n_zero, res.n_keep) == (r.n_units, r.n_zero, r.n_keep)
        assert res.tau_id == r.tau_id
        assert (res.n_gt, res.n_tie, res.n_tie_kept) == (r.n_gt, r.n_tie, r.n_tie_kept)
        if exact_key:
            assert res.tau_key == r.tau_key
        else:   # filter norms: the fp64 summation order differs from the oracle's
            a = np.array([res.tau_key], np.uint64).view(np.float64)[0]
            b = np.array([r.tau_key], np.uint64).view(np.float64)[0]
            assert a == b or abs(a - b) <= 1e-12 * abs(b)
        if op != "prune" and r.n_keep > 0:
            assert abs(res.tau_norm - r.tau_norm) <= REL * abs(r.tau_norm)
    return got, res, exp


# ---------------------------------------------------------------- elementwise
@pytest.mark.parametrize("n", [1, 3, 4, 5, 1023, 4096, 4097, 100003])
@pytest.mark.parametrize("off", [0, 1, 2, 3])
def test_quantize_sizes_and_alignments(ctx, n, off):
    ws = W.random_set([(n,)], seed=n + off, kind="normal", scale=3.0, lam_sigma=1e-2, mu=1e-2)
    check(ctx, "quantize", ws.w, ws.lam, mu=ws.mu, fuse=("lambda", "penalty"), elem_offset=off)


def test_quantize_special_values_and_skewed_alignment(ctx):
    sp = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, -np.nan, 65504.0, 65519.99, 65520.0, 1e-8,
                   2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001, 6.1e-5, -6.0e-8, 1e-45, 3.4e38],
                  np.float32)
    w = np.tile(sp, 40)
    got, _, exp = check(ctx, "quantize", [w], [None], mu=1.0, fuse=())
    # no arithmetic touches u here, so even the NaN signs must come through
    assert np.array_equal(got["theta_h"][0], exp.theta_h[0])
    check(ctx, "quantize", [w], [np.zeros_like(w)], mu=1.0, fuse=("lambda", "penalty"), skew=1)
    ws = W.random_set([(7, 9), (5,), (2, 3, 4, 5)], seed=3, kind="normal", scale=100.0, lam_sigma=1.0, mu=0.5)
    check(ctx, "quantize", ws.w, ws.lam, mu=ws.mu, fuse=("penalty",), elem_offset=1, skew=2)


def test_bf16_quantize_and_fused_paths(ctx):
    sp = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, -np.nan, 1.0, 1.00390625, 1.01171875, 3.3895314e38,
                   3.38e38, 1e-40, -1e-45, 0.1, 65504.0], np.float32)
    got, _, exp = check(ctx, "quantize_bf16", [np.tile(sp, 300)], [None], mu=1.0, fuse=())
    assert np.array_equal(got["theta_h"][0], exp.theta_h[0])
    for n, off in ((5, 0), (4099, 1), (100003, 3)):
        ws = W.random_set([(n,)], seed=n, kind="normal", scale=3.0, lam_sigma=1e-2, mu=1e-2)
        check(ctx, "quantize_bf16", ws.w, ws.lam, mu=ws.mu, fuse=("lambda", "penalty"), elem_offset=off)
    ws = W.config(4, scale=0.1)                               # single-pass path with bfloat16
    check(ctx, "prune", ws.w, ws.lam, ws.sparsity, ws.mu, ("bf16", "lambda", "penalty"))
    check(ctx, "prune", ws.w, ws.lam, ws.sparsity, ws.mu, ("bf16", "lambda", "no_sampling"))
    ws = W.config("5", scale=0.12)
    check(ctx, "block", ws.w, ws.lam, ws.sparsity, ws.mu, ("bf16", "lambda"))
    check(ctx, "block", ws.w, ws.lam, ws.sparsity, ws.mu, ("bf16", "lambda"), block=(5, 5))
    ws = W.config(3, scale=0.2)
    check(ctx, "filter", ws.w, ws.lam, ws.sparsity, ws.mu, ("bf16", "lambda"), exact_key=False)
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ds = DeviceSet(ws.w, ws.lam)
    with pytest.raises(cstep.CondensaError):
        ds.run(ctx, "prune", 0.5, 1e-3, ("fp16", "bf16"))


@pytest.mark.parametrize("dtype", ["fp16", "bf16", "e4m3", "e5m2"])
def test_quantize_every_fp32_bit_pattern(ctx, dtype):
    """All 2^32 binary32 patterns through the quantise entry point against the oracle's
    explicit-bit conversion (the code and the widened theta)."""
    import torch
    from paper_1911_02497_b200 import cstep
    chunk = 1 << 27
    dev = torch.device("cuda:0")
    w = torch.empty(chunk, dtype=torch.int32, device=dev)
    theta = torch.empty(chunk, dtype=torch.float32, device=dev)
    th = torch.empty(chunk, dtype=torch.int16, device=dev)
    base = torch.arange(chunk, dtype=torch.int64, device=dev)
    tab = cstep.tensor_table([w], None, [theta], None, None, [th], shapes=[(chunk,)])
    code = {"fp16": cstep.DTYPE_FP16, "bf16": cstep.DTYPE_BF16, "e4m3": cstep.DTYPE_FP8_E4M3,
            "e5m2": cstep.DTYPE_FP8_E5M2}[dtype]
    tdt = {"fp16": torch.float16, "bf16": torch.bfloat16, "e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}[dtype]
    eight = dtype in ("e4m3", "e5m2")
    for c in range((1 << 32) // chunk):
        first = c * chunk
        w.copy_(((base + first) & 0xFFFFFFFF).to(torch.int64).sub_((base + first >= (1 << 31)).to(torch.int64) << 32).to(torch.int32))
        ctx.cstep_quantize(tab, 1, 1.0, dtype=code)
        got_h = th.cpu().numpy().view(np.uint16)
        if eight:
            exp8 = oracle.f32_to_fp8_range(first, chunk, dtype)
            exp_h = exp8.astype(np.uint16)
        else:
            exp_h = (oracle.f32_to_f16_range if dtype == "fp16" else oracle.f32_to_bf16_range)(first, chunk)
        assert np.array_equal(got_h, exp_h), "chunk %d" % c
        # theta is the exact widening of that code (NaN: quiet, sign kept); torch's widening is exact
        src = torch.from_numpy(exp8.copy()).to(dev) if eight else torch.from_numpy(exp_h.view(np.int16)).to(dev)
        wide = src.view(tdt).to(torch.float32)
        tb, wb = theta.view(torch.int32), wide.view(torch.int32)
        nan = torch.isnan(wide)
        assert bool(torch.equal(tb[~nan], wb[~nan]))
        neg = torch.from_numpy((exp_h >> (7 if eight else 15)).astype(np.bool_)).to(dev)
        assert bool(torch.isnan(theta[nan]).all()) and bool(torch.equal(tb[nan] < 0, neg[nan]))    # sign kept
    torch.cuda.synchronize()


@pytest.mark.parametrize("q", ["e4m3", "e5m2"])
def test_eight_bit_types_in_the_fused_paths(ctx, q):
    """Compose([Prune, Quantize(8-bit)]) and the structured schemes with an 8-bit type: two-pass
    sizes, single-pass sizes (elements and 4x4 blocks), filters, with multipliers and gradient."""
    ws = W.random_set([(33, 17), (4099,), (5, 3, 3, 3)], seed=9, kind="normal", scale=2.0, lam_sigma=1e-2, mu=1e-2)
    check(ctx, "quantize_" + q, ws.w, ws.lam, mu=ws.mu, fuse=("lambda", "penalty"), elem_offset=1)
    check(ctx, "prune", ws.w, ws.lam, 0.7, ws.mu, (q, "lambda", "penalty"))
    check(ctx, "filter", ws.w, ws.lam, 0.4, ws.mu, (q, "lambda"), exact_key=False)
    check(ctx, "block", ws.w, ws.lam, 0.5, ws.mu, (q, "lambda"))
    big = W.random_set([(1300000,), (270001,)], seed=10, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    got, res, _ = check(ctx, "prune", big.w, big.lam, 0.9, big.mu, (q, "lambda", "penalty"))
    assert res.sampled == 1
    m = W.random_set([(1600, 1000), (602, 1000)], seed=11, kind="uniform", scale=0.1, lam_sigma=1e-3, mu=1e-2)
    got, res, _ = check(ctx, "block", m.w, m.lam, 0.9, m.mu, (q, "lambda", "penalty"))
    assert res.sampled == 1


@pytest.mark.parametrize("fuse", [("lambda",), ("penalty",), ("lambda", "penalty")])
def test_lagrange_update(ctx, fuse):
    ws = W.random_set([(33, 17), (4096,), (5, 3, 3, 3), (1,)], seed=8, kind="normal", scale=0.1,
                      lam_sigma=1e-2, mu=1e-2)
    th = [np.where(np.abs(a) > 0.08, a, 0).astype(np.float32) for a in ws.w]
    got, _, exp = check(ctx, "lagrange", ws.w, ws.lam, mu=ws.mu, fuse=fuse, theta=th)
    if "lambda" not in fuse:
        for t in range(4):
            assert np.array_equal(bits(got["lam"][t]), bits(ws.lam[t]))   # untouched
    check(ctx, "lagrange", ws.w, [None] * 4, mu=ws.mu, fuse=fuse, theta=th, elem_offset=3)
    # w == theta leaves lambda bit-identical and zero stays zero
    got, _, _ = check(ctx, "lagrange", ws.w, [np.zeros_like(a) for a in ws.w], mu=ws.mu,
                      fuse=("lambda",), theta=[a.copy() for a in ws.w])
    assert all(np.all(bits(x) == 0) for x in got["lam"])


# ---------------------------------------------------------------- unstructured
@pytest.mark.parametrize("n,s", [(1, 0.0), (1, 1.0), (2, 0.5), (7, 0.5), (100, 0.01), (100, 0.99),
                                 (4096, 0.9), (4099, 0.37), (70001, 0.95), (300007, 0.5)])
def test_prune_small(ctx, n, s):
    ws = W.random_set([(n,)], seed=n, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    check(ctx, "prune", ws.w, ws.lam, s, ws.mu, ("lambda", "penalty"))


@pytest.mark.parametrize("off,skew", [(1, 0), (2, 0), (3, 0), (0, 1), (1, 2)])
def test_prune_unaligned(ctx, off, skew):
    ws = W.random_set([(5003,), (17, 13), (4, 3, 3, 3)], seed=off * 7 + skew, kind="normal",
                      scale=0.05, lam_sigma=1e-2, mu=1e-2)
    check(ctx, "prune", ws.w, ws.lam, 0.8, ws.mu, ("fp16", "lambda", "penalty"), elem_offset=off, skew=skew)


def test_prune_ties_and_degenerate_inputs(ctx):
    n = 300000          # larger than the candidate list: ties must be settled by index passes
    check(ctx, "prune", [np.full(n, 0.5, np.float32)], None, 0.7, 1.0, ())
    check(ctx, "prune", [np.zeros(n, np.float32)], None, 0.25, 1.0, ("lambda",))
    two = np.where(np.arange(n) % 3 == 0, 1.0, -0.25).astype(np.float32)
    check(ctx, "prune", [two], None, 0.5, 1.0, ())          # threshold inside the big tie group
    check(ctx, "prune", [two], None, 0.8, 1.0, ())          # threshold inside the small one
    pm = np.tile(np.array([1.0, -1.0, 0.0, -0.0], np.float32), 1000)
    check(ctx, "prune", [pm], None, 0.6, 1.0, ())
    a = np.array([2.0, 1.0], np.float32); b = np.array([1.0, 1.0, 3.0], np.float32)
    check(ctx, "prune", [a, b], None, 0.4, 1.0, ())         # tie across a tensor boundary
    w = np.array([1.0, np.inf, np.nan, -np.inf, 0.5], np.float32)
    check(ctx, "prune", [w], None, 0.6, 1.0, ())
    den = (np.arange(1, 2001, dtype=np.uint32) * 4099 % 8388607).view(np.float32)   # subnormals
    check(ctx, "prune", [den], None, 0.5, 1.0, ())
    q = np.round(W.draw(500000, "normal", 4.0, 1, 0, 0)).astype(np.float32)         # few distinct values
    check(ctx, "prune", [q], None, 0.9, 1.0, ("lambda",))


def test_edge_sparsities_at_single_pass_sizes(ctx):
    """Sizes that go for the single pass, with the sparsities at which it must step aside or
    work at the very ends of the ranking: nothing pruned, everything pruned, one unit pruned,
    one unit kept. With 16-bit output, so that the projection a fall-back makes inside the
    selection kernel writes the codes too."""
    n = 400000
    w = W.draw(n, "normal", 0.05, 71, 0, 0)
    lam = W.draw(n, "normal", 0.01, 71, 1, 0)
    for s in (0.0, 1.0, 1.0 / n, 1.0 - 1.0 / n):
        check(ctx, "prune", [w[:150000], w[150000:]], [lam[:150000], lam[150000:]], s, 1e-2, ("fp16", "lambda", "penalty"))
    m = W.draw(600 * 1000, "uniform", 0.1, 72, 0, 0).reshape(600, 1000)        # 37500 blocks
    big = W.draw(2400 * 1000, "uniform", 0.1, 73, 0, 0).reshape(2400, 1000)    # 150000 blocks: together a single-pass size
    nb = 150000 + 37500
    for s in (0.0, 1.0, 1.0 / nb, 1.0 - 1.0 / nb):
        check(ctx, "block", [big, m, np.ones(7, np.float32)], None, s, 1e-3, ("bf16", "lambda"))
    # a tie group far larger than the candidate list: the sample advises against the single pass
    ties = np.where(np.arange(n) % 2 == 0, 0.25, -0.25).astype(np.float32)
    check(ctx, "prune", [ties], None, 0.5, 1.0, ("fp16", "lambda"))


def test_prune_k_zero_keep_all_and_empty_tensors(ctx):
    ws = W.random_set([(1000,), (0,), (37,)], seed=1, kind="normal", scale=1.0)
    for s in (0.0, 1.0, 1e-9, 1 - 1e-9):
        check(ctx, "prune", ws.w, None, s, 1.0, ("lambda", "penalty"))


def test_prune_idempotent_and_unfused_sequence(ctx):
    ws = W.config(2, scale=0.3)
    got, res, _ = check(ctx, "prune", ws.w, ws.lam, 0.95, ws.mu, ("fp16", "lambda"))
    again, _ = run_gpu(ctx, "prune", got["theta"], [None] * len(ws.w), 0.95, 1.0, ())
    for a, b in zip(got["theta"], again["theta"]):
        assert np.array_equal(bits(a), bits(b))
    # unfused: prune, quantise theta, multiplier update == fused call
    p, _ = run_gpu(ctx, "prune", ws.w, ws.lam, 0.95, ws.mu, ())
    q, _ = run_gpu(ctx, "quantize", p["theta"], [None] * len(ws.w), 0.0, ws.mu, ())
    l, _ = run_gpu(ctx, "lagrange", ws.w, ws.lam, 0.0, ws.mu, ("lambda",), theta=q["theta"])
    for t in range(len(ws.w)):
        assert np.array_equal(p["mask"][t], got["mask"][t])
        assert np.array_equal(bits(q["theta"][t]), bits(got["theta"][t]))
        assert np.array_equal(bits(l["lam"][t]), bits(got["lam"][t]))


@pytest.mark.parametrize("cfg,scale", [(1, 1.0), (2, 1.0), (4, 0.12)])
def test_prune_configurations(ctx, cfg, scale):
    ws = W.config(cfg, scale=scale)
    got, res, _ = check(ctx, "prune", ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse)
    zeros = sum(int((m == 0).sum()) for m in got["mask"])
    assert zeros == res.n_zero == math.floor(ws.sparsity * ws.numel + 0.5)


@pytest.mark.parametrize("cfg,scale", [(1, 1.0), (2, 1.0), (4, 0.12), ("5", 0.1)])
def test_two_pass_path_without_sampling(ctx, cfg, scale):
    """The same configurations with the sample bracket switched off: rank first
    (full histogram passes), then project."""
    ws = W.config(cfg, scale=scale)
    got, res, _ = check(ctx, ws.op, ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse + ("no_sampling",))
    assert res.sampled == 0 and res.n_repaired == 0


def test_single_pass_path_is_taken_and_repairs(ctx):
    ws = W.random_set([(1 << 21,)], seed=0, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)     # too long for the registers
    got, res, _ = check(ctx, "prune", ws.w, ws.lam, 0.9, ws.mu, ("fp16", "lambda"))
    assert res.sampled == 1 and 0 < res.n_candidates < ws.numel // 8
    ws = W.config("5", scale=0.2)
    got, res, _ = check(ctx, "block", ws.w, ws.lam, ws.sparsity, ws.mu, ("fp16", "lambda", "penalty"))
    assert res.sampled == 1 and 0 < res.n_candidates < res.n_units // 8


def _adversarial_for_seed(seed, n=3 << 19, m=16384):
    """An input built against the sample positions of `seed`: tiny values exactly there, so that
    the bracket taken from the sample cannot hold the threshold of the whole tensor."""
    w = W.draw(n, "normal", 1.0, 77, 0, 0)
    pos = [(W._mix64_scalar(W._mix64_scalar(seed) ^ j) * n) >> 64 for j in range(m)]
    w[np.array(pos)] = W.draw(m, "normal", 1e-4, 78, 0, 0)
    return w


def test_sample_bracket_miss_falls_back_or_is_reported(ctx):
    """The single-pass path trusts a bracket taken from 16384 hashed positions and checks it
    exactly afterwards. With an input built against the positions of a known seed the bracket
    misses. When the first pass has not overwritten multipliers the call must fall back by
    itself and return the oracle's result; with in-place multipliers it must say so through the
    result status instead of returning a wrong projection; with any other seed the same input
    goes through the single pass; and the context must stay usable throughout."""
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    seed = 0x9E3779B97F4A7C15
    w = _adversarial_for_seed(seed)
    lam = W.draw(w.size, "normal", 1e-4, 79, 1, 0)
    try:
        ctx.set_seed(seed)
        # no multiplier is updated: falls back inside the call, exact result, not sampled
        for fuse, l in ((("penalty", "fp16"), [lam]), (("lambda",), [None]), ((), [lam])):
            got, res, _ = check(ctx, "prune", [w], l, 0.9, 1e-3, fuse)
            assert res.sampled == 0 and res.n_repaired == 0 and res.seed == seed
        # multipliers updated in place: reported, never silent
        ds = DeviceSet([w], [lam])
        ds.run(ctx, "prune", 0.9, 1e-3, ("lambda",))
        with pytest.raises(cstep.CondensaError) as e:
            ctx.get_result()
        assert e.value.code == cstep.ERR_INTERNAL
        # another seed: the same input and call succeed on the single pass
        ctx.set_seed(seed + 12345)
        got, res, _ = check(ctx, "prune", [w], [lam], 0.9, 1e-3, ("lambda",))
        assert res.sampled == 1 and res.seed == seed + 12345
        # and without the sample bracket it is projected correctly whatever the seed
        ctx.set_seed(seed)
        check(ctx, "prune", [w], [lam], 0.9, 1e-3, ("lambda", "no_sampling"))
    finally:
        ctx.set_seed(SEED)


def test_more_candidates_than_the_list_holds_falls_back(ctx):
    """A tie group that the sample cannot see but that overflows the candidate list: the values at
    the sampled positions are spread out, everything else within the bracket is one value."""
    seed = 0x1234ABCD
    n, m = 3 << 19, 16384
    w = np.full(n, 0.5, np.float32)
    w[::20] = 2.0                                    # 5 % clearly above the cut of s = 0.9
    pos = np.array([(W._mix64_scalar(W._mix64_scalar(seed) ^ j) * n) >> 64 for j in range(m)])
    w[pos] = W.draw(m, "uniform", 0.5 / 0.9, 80, 0, 0)   # the sample sees |u| spread evenly, 10 % above 0.5
    try:
        ctx.set_seed(seed)
        for fuse in (("penalty",), ("fp16",)):
            got, res, _ = check(ctx, "prune", [w], [np.zeros_like(w)], 0.9, 1e-3, fuse)
            assert res.sampled == 0 and res.n_tie > 1400000
    finally:
        ctx.set_seed(SEED)


def test_single_pass_with_and_without_multipliers_in_one_list(ctx):
    """Tensors with and without a lambda buffer in one sampled call: the journal of a candidate
    must carry the multiplier of its own tensor (candidates staged by one tensor are flushed
    while the CTA already works on the next)."""
    shapes = [(280001,), (200000,), (493457,), (4099,), (800003,)]
    ws = W.random_set(shapes, seed=91, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    lam = [ws.lam[0], None, ws.lam[2], None, ws.lam[4]]
    for sd in (1, 2, 3):
        ctx.set_seed(sd)
        got, res, _ = check(ctx, "prune", ws.w, lam, 0.9, ws.mu, ("fp16", "lambda", "penalty"))
        assert res.sampled == 1 and res.n_repaired > 0
        got, res, _ = check(ctx, "prune", ws.w, lam, 0.9, ws.mu, ("lambda",), elem_offset=1)
        assert res.sampled == 1
    ctx.set_seed(SEED)


def test_result_record_of_the_one_cta_selection(ctx):
    """The record a short ranking leaves: passes, counts and cut-off as the oracle has them."""
    ws = W.random_set([(300, 64)], seed=3, kind="normal", scale=1.0)
    got, res, exp = check(ctx, "neuron", ws.w, None, 0.5, 1.0, (), exact_key=False)
    assert res.passes >= 1 and res.n_candidates == 300 and res.sampled == 0 and res.n_repaired == 0


# ---------------------------------------------------------------- filters
def test_filter_small_and_ties(ctx):
    ws = W.random_set([(7, 3, 3, 3), (10, 12), (9, 7, 1, 1), (6, 300, 3, 3), (3,)], seed=2,
                      kind="normal", scale=0.2, lam_sigma=1e-2, mu=1e-2)
    for s in (0.0, 0.3, 0.6, 1.0):
        check(ctx, "filter", ws.w, ws.lam, s, ws.mu, ("lambda", "penalty"), exact_key=False)
    check(ctx, "filter", ws.w, ws.lam, 0.5, ws.mu, ("fp16", "lambda"), elem_offset=1, exact_key=False)
    f = W.draw(2 * 5 * 9, "normal", 1.0, 5, 0, 0).reshape(2, 5, 3, 3)
    dup = np.concatenate([f, f, f], 0)                        # filters 0,2,4 and 1,3,5 identical
    got, res, _ = check(ctx, "filter", [dup], None, 0.5, 1.0, (), exact_key=False)
    assert res.n_tie == 3
    ints = np.round(W.draw(8 * 3000, "normal", 3.0, 6, 0, 0)).reshape(8, 3000, 1, 1).astype(np.float32)
    check(ctx, "filter", [ints, ints[::-1].copy()], None, 0.5, 1.0, ())   # integer data: sums exact
    check(ctx, "filter", [np.ones((4, 5), np.float32)], None, 0.5, 1.0, ())   # nothing to rank


@pytest.mark.parametrize("op", ["neuron", "structure"])
def test_neuron_and_structure_pruning(ctx, op):
    """Rows of 2-D tensors (NeuronPrune) and rows + filters in one ranking (StructurePrune)."""
    ws = W.random_set([(300, 257), (7, 3, 3, 3), (64,), (40, 1024), (12, 20, 3, 3), (1, 9)], seed=44,
                      kind="normal", scale=0.3, lam_sigma=1e-2, mu=1e-2)
    for s in (0.0, 0.35, 0.8, 1.0):
        check(ctx, op, ws.w, ws.lam, s, ws.mu, ("lambda", "penalty"), exact_key=False)
    check(ctx, op, ws.w, ws.lam, 0.5, ws.mu, ("fp16", "lambda"), elem_offset=3, exact_key=False)
    # LSTM-shaped set: rows of the big matrices
    ws = W.config("5t", scale=0.1)
    got, res, _ = check(ctx, op, ws.w, ws.lam, 0.6, ws.mu, ("lambda",), exact_key=False)
    assert res.n_units == sum(a.shape[0] for a in ws.w if a.ndim == 2)


@pytest.mark.parametrize("extra", [(), ("no_sampling",)])
def test_short_rankings_one_cta_and_general_selection_agree(ctx, extra):
    """Rankings of at most 16384 structures run in one CTA; `no_sampling` forces the
    grid-wide selection. Both must give the oracle's result: many equal norms (ties
    settled by index), every rank from the first to the last, k = 0 and k = S, and a
    ranking just below and just above the one-CTA limit."""
    rng = np.random.default_rng(9)
    vals = rng.integers(1, 6, size=700).astype(np.float32)        # few distinct norms: long ties
    rows = np.repeat(vals[:, None], 8, axis=1) * np.where(rng.random((700, 8)) < 0.5, -1, 1).astype(np.float32)
    for s in (0.0, 1 / 700, 0.31, 0.5, 0.77, 1 - 1 / 700, 1.0):
        got, res, exp = check(ctx, "neuron", [rows], None, s, 1.0, tuple(extra))
    assert res.n_units == 700
    # blocks of a general shape: 5 x 5 blocks of a 200 x 300 matrix (2400 units), with lambda
    ws = W.random_set([(200, 300), (64,)], seed=12, kind="normal", scale=0.2, lam_sigma=1e-2, mu=1e-2)
    check(ctx, "block", ws.w, ws.lam, 0.6, ws.mu, ("lambda",) + tuple(extra), block=(5, 5))
    # around the limit: 16384 and 16385 rows
    for n in (16384, 16385):
        m = W.draw(n * 4, "normal", 1.0, 13, 0, 0).reshape(n, 4)
        got, res, _ = check(ctx, "neuron", [m], None, 0.9, 1.0, tuple(extra), exact_key=False)
        assert res.n_units == n


@pytest.mark.parametrize("scale", [0.25, 1.0])
def test_filter_configuration(ctx, scale):
    ws = W.config(3, scale=scale)
    nu = oracle.structure_norms(ws.w, ws.lam, ws.mu, "filter")
    srt = np.sort(nu)[::-1]
    k = nu.size - oracle.round_count(ws.sparsity, nu.size)
    assert (srt[k - 1] - srt[k]) > 1e-9 * srt[k - 1]          # kept set is decided well above fp64 noise
    check(ctx, "filter", ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse, exact_key=False)


# ---------------------------------------------------------------- blocks
@pytest.mark.parametrize("shape", [(4, 4), (1, 1), (3, 5), (8, 12), (10, 14), (33, 28), (64, 1500 // 4 * 4 + 2),
                                   (130, 256)])
def test_block_shapes(ctx, shape):
    ws = W.random_set([shape, (11,), (shape[1], shape[0])], seed=sum(shape), kind="uniform", scale=0.1,
                      lam_sigma=1e-3, mu=1e-2)
    for s in (0.0, 0.5, 0.9, 1.0):
        check(ctx, "block", ws.w, ws.lam, s, ws.mu, ("lambda", "penalty"))
    check(ctx, "block", ws.w, ws.lam, 0.7, ws.mu, ("fp16", "lambda"), elem_offset=2)
    check(ctx, "block", ws.w, ws.lam, 0.7, ws.mu, ("lambda",), skew=1)


@pytest.mark.parametrize("block", [(5, 5), (1, 8), (3, 2), (8, 1), (16, 16), (2, 4)])
def test_block_general_shapes(ctx, block):
    """Block sizes other than 4x4 (the paper's LSTM experiment uses bs = 5)."""
    ws = W.random_set([(33, 28), (11,), (130, 257), (5, 5), (64, 1500)], seed=sum(block), kind="uniform",
                      scale=0.1, lam_sigma=1e-3, mu=1e-2)
    for s in (0.0, 0.6, 1.0):
        check(ctx, "block", ws.w, ws.lam, s, ws.mu, ("lambda", "penalty"), block=block)
    check(ctx, "block", ws.w, ws.lam, 0.9, ws.mu, ("fp16", "lambda"), block=block, elem_offset=1)
    blk = np.arange(block[0] * block[1], dtype=np.float32).reshape(block)
    got, res, _ = check(ctx, "block", [np.tile(blk, (3, 4))], None, 0.5, 1.0, (), block=block)   # 12 equal blocks
    assert (res.n_tie, res.n_tie_kept) == (12, 6)


def test_single_pass_block_kernel_tiles_edges_and_many_tensors(ctx):
    """The tiled single-pass block kernel at a size that takes it (more than 131072 blocks):
    more tensors than its descriptor cache holds, block rows that are no multiple of the tile
    width, ragged last block rows, a matrix whose width is no multiple of 4 and a vector (both
    done by the generic code), then the same list on buffers that are not 16-byte aligned."""
    shapes = [(130, 1000)] * 17 + [(66, 1001), (4097,), (64, 32), (4, 128)]
    ws = W.random_set(shapes, seed=77, kind="uniform", scale=0.1, lam_sigma=1e-3, mu=1e-2)
    for sd in (5, 6):
        ctx.set_seed(sd)
        got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.9, ws.mu, ("lambda", "penalty"))
        assert res.sampled == 1 and res.n_units > 131072 and res.n_candidates > 0
    got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.5, ws.mu, ("fp16", "lambda"))
    assert res.sampled == 1
    lam = [l if t % 3 else None for t, l in enumerate(ws.lam)]
    got, res, _ = check(ctx, "block", ws.w, lam, 0.8, ws.mu, ("bf16", "lambda", "penalty"))
    assert res.sampled == 1
    got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.9, ws.mu, ("lambda",), elem_offset=2)
    assert res.sampled == 1
    ctx.set_seed(SEED)


@pytest.mark.parametrize("block", [(5, 5), (3, 3), (1, 8), (8, 1), (2, 2), (3, 2), (7, 3)])
def test_single_pass_general_blocks(ctx, block):
    """bh x bw blocks at a size that takes the tiled single-pass kernel (more than 131072 blocks):
    several block rows per tile and one per tile, ragged last block rows, widths that are no
    multiple of bw, a matrix whose width is no multiple of 4, a vector and a 4-D tensor (pass
    through), tensors without multipliers, 16-bit codes and gradient. The kernel is built for the
    first five shapes; the others take the route over the norm array at the same size."""
    bh, bw = block
    tiled = 1 if block in ((5, 5), (3, 3), (1, 8), (8, 1), (2, 2)) else 0
    shapes = [(bh * 37 + bh // 2, 1500), (203 * bh, 8 * bw * 4), (61, 1001), (4097,), (401, 1204), (3, 2, 4, 4),
              (bh + 1, 1024 * bw)]
    need = 140000 * bh * bw - sum(r * c for r, c in [sh for sh in shapes if len(sh) == 2])
    shapes.append((max(need // 1000 + 1, bh), 1000))
    ws = W.random_set(shapes, seed=31 + bh * 9 + bw, kind="uniform", scale=0.1, lam_sigma=1e-3, mu=1e-2)
    for sd in (5, 6):
        ctx.set_seed(sd)
        got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.9, ws.mu, ("lambda", "penalty"), block=block)
        assert res.sampled == tiled and res.n_units > 131072
        assert not tiled or (res.n_candidates > 0 and res.n_repaired > 0)
    got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.5, ws.mu, ("fp16", "lambda"), block=block)
    assert res.sampled == tiled
    lam = [l if t % 3 else None for t, l in enumerate(ws.lam)]
    got, res, _ = check(ctx, "block", ws.w, lam, 0.8, ws.mu, ("bf16", "lambda", "penalty"), block=block)
    assert res.sampled == tiled
    got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.9, ws.mu, (), block=block)     # nothing updated in place
    assert res.sampled == tiled
    ctx.set_seed(SEED)


def test_block_shapes_alternate_on_one_context(ctx):
    """One context serves 4 x 4, 5 x 5 and 2 x 2 block calls and an unstructured call in turn, at sizes
    that take the single-pass kernels: workspace layout, descriptor cache and shared-memory
    configuration change from call to call."""
    ws = W.random_set([(2500, 1200), (803, 1000), (77,), (1000, 640)], seed=91, kind="uniform", scale=0.1,
                      lam_sigma=1e-3, mu=1e-2)
    # (2 x 2 at s = 0.7: the sample's bracket would hold more blocks than the list takes, so the
    # selection kernel does the two-pass job for that call)
    for block, s, single in (((4, 4), 0.9, 1), ((5, 5), 0.9, 1), ((2, 2), 0.7, 0), ((5, 5), 0.5, 1), ((2, 2), 0.9, 1),
                             ((4, 4), 0.6, 1)):
        got, res, _ = check(ctx, "block", ws.w, ws.lam, s, ws.mu, ("lambda",), block=block)
        assert res.sampled == single, block
        got, res, _ = check(ctx, "prune", ws.w, ws.lam, 0.8, ws.mu, ("lambda", "penalty"))
        assert res.sampled == 1


def test_single_pass_general_blocks_fall_back(ctx):
    """A list whose block norms are nearly all equal: the sample advises against the single pass and
    the selection kernel does the two-pass job for bh x bw blocks itself."""
    rng = np.random.default_rng(12)
    w = [np.full((3000, 1500), 0.25, np.float32), rng.standard_normal((100, 200)).astype(np.float32)]
    got, res, _ = check(ctx, "block", w, None, 0.5, 1e-2, ("penalty",), block=(5, 5))
    assert res.sampled == 0 and res.n_units == 600 * 300 + 20 * 40


def check_structured(ctx, w, lam, s, mu, kind, block=None, criterion="l2", fuse=("lambda",), elem_offset=0,
                     exact_key=True):
    """The specification entry point against the oracle's: masks, theta, multipliers, gradient and
    the record; the ranked value bit for bit where the summation order is the definition's."""
    from paper_1911_02497_b200.device_set import DeviceSet
    lam = lam if lam is not None else [None] * len(w)
    ds = DeviceSet(w, lam, elem_offset=elem_offset)
    ds.poison_outputs()
    ctx.cstep_structured(ds.table, ds.T, s, mu, kind, block, criterion, fuse)
    got, res = ds.fetch(), ctx.get_result()
    exp = oracle.cstep_structured(w, lam, s, mu, kind, block, criterion, tuple(f for f in fuse if f != "no_sampling"))
    for t in range(len(w)):
        assert np.array_equal(got["mask"][t], exp.mask[t]), "mask, tensor %d" % t
        assert same_f32(got["theta"][t], exp.theta[t]), "theta, tensor %d" % t
        if lam[t] is not None:
            assert same_f32(got["lam"][t], exp.lam[t]), "lambda, tensor %d" % t
        if "penalty" in fuse:
            assert same_f32(got["grad"][t], exp.grad[t]), "grad, tensor %d" % t
    r = exp.result
    assert res.status == 0 and (res.n_units, res.n_zero, res.n_keep, res.tau_id) == (r.n_units, r.n_zero, r.n_keep, r.tau_id)
    assert (res.n_gt, res.n_tie, res.n_tie_kept) == (r.n_gt, r.n_tie, r.n_tie_kept)
    if exact_key:
        assert res.tau_key == r.tau_key
    else:
        a, b = (np.array([k], np.uint64).view(np.float64)[0] for k in (res.tau_key, r.tau_key))
        assert a == b or abs(a - b) <= 1e-12 * abs(b)
    if r.n_keep > 0:
        assert abs(res.tau_norm - r.tau_norm) <= REL * abs(r.tau_norm)
    return got, res, exp


@pytest.mark.parametrize("crit", ["l2", "l1", "max"])
def test_structure_criteria(ctx, crit):
    """Filters, neurons, both, and 2-D blocks ranked by the L2, L1 or max criterion."""
    ws = W.random_set([(300, 257), (7, 3, 3, 3), (64,), (40, 1024), (12, 20, 3, 3), (1, 9)], seed=45,
                      kind="normal", scale=0.3, lam_sigma=1e-2, mu=1e-2)
    for kind in ("filter", "neuron", "structure"):
        for s in (0.0, 0.4, 1.0):
            check_structured(ctx, ws.w, ws.lam, s, ws.mu, kind, None, crit, ("lambda", "penalty"), exact_key=(crit == "max"))
    check_structured(ctx, ws.w, ws.lam, 0.7, ws.mu, "structure", None, crit, ("fp16", "lambda"), elem_offset=3,
                     exact_key=(crit == "max"))
    for block in ((5, 5), (4, 4), (1, 8)):
        check_structured(ctx, ws.w, ws.lam, 0.6, ws.mu, "block", block, crit, ("lambda",))
    # many equal values: ties settled by the structure index, in one CTA and grid-wide
    rows = np.tile(np.array([[1.0, -2.0, 0.5, 2.0]], np.float32), (900, 1)) * np.repeat(
        np.arange(1, 4, dtype=np.float32), 300)[:, None]
    for extra in ((), ("no_sampling",)):
        got, res, _ = check_structured(ctx, [rows], None, 0.5, 1.0, "neuron", None, crit, extra)
        assert res.n_tie == 300
    # the VGG-shaped set: the filter ranking with the other criteria
    ws = W.config(3, scale=0.25)
    check_structured(ctx, ws.w, ws.lam, 0.8, ws.mu, "filter", None, crit, ("lambda",), exact_key=(crit == "max"))


@pytest.mark.parametrize("block", [(2, 2, 2), (1, 3, 2), (2, 1, 3, 3), (3, 2, 1, 2), (5,), (4, 4), (7, 3)])
def test_nd_blocks(ctx, block):
    """BlockPrune with n-D blocks: tensors of that rank are cut, the others pass through."""
    nd = len(block)
    shape = {1: (10007,), 2: (129, 70), 3: (33, 17, 9), 4: (20, 9, 5, 5)}[nd]
    other = {1: (4, 4), 2: (6,), 3: (6, 5), 4: (7, 2, 2)}[nd]
    ws = W.random_set([shape, other, shape, (5,) * nd], seed=50 + nd, kind="normal", scale=0.3, lam_sigma=1e-2, mu=1e-2)
    for s in (0.0, 0.45, 0.9, 1.0):
        check_structured(ctx, ws.w, ws.lam, s, ws.mu, "block", block, "l2", ("lambda", "penalty"))
    check_structured(ctx, ws.w, ws.lam, 0.5, ws.mu, "block", block, "l1", ("bf16", "lambda"), elem_offset=1)
    check_structured(ctx, ws.w, ws.lam, 0.5, ws.mu, "block", block, "max", ("lambda", "no_sampling"))


def test_conv_weights_in_3d_blocks_at_size(ctx):
    """3-D blocks over conv weights of a VGG-shaped set seen as [F, C, kh*kw] (more than 16384 blocks:
    the grid-wide selection on the value array)."""
    ws = W.config(3, scale=0.25)
    w = [a.reshape(a.shape[0], a.shape[1], -1) if a.ndim == 4 else a for a in ws.w]
    lam = [l.reshape(a.shape) for l, a in zip(ws.lam, w)]
    got, res, _ = check_structured(ctx, w, lam, 0.7, ws.mu, "block", (2, 2, 9), "l2", ("lambda",))
    assert res.n_units > 16384


def test_block_size_five_on_the_lstm_shapes(ctx):
    ws = W.config("5", scale=0.1)
    got, res, _ = check(ctx, "block", ws.w, ws.lam, 0.6, ws.mu, ("lambda",), block=(5, 5))
    assert res.n_units == sum(-(-a.shape[0] // 5) * -(-a.shape[1] // 5) for a in ws.w if a.ndim == 2)


def test_block_ties(ctx):
    blk = np.arange(16, dtype=np.float32).reshape(4, 4)
    got, res, _ = check(ctx, "block", [np.tile(blk, (2, 3))], None, 0.5, 1.0, ())
    assert (res.n_tie, res.n_tie_kept, res.tau_id) == (6, 3, 2)
    big = np.tile(blk, (600, 300))                            # 180000 equal blocks
    check(ctx, "block", [big], None, 0.9, 1.0, ("lambda",))
    check(ctx, "block", [np.zeros((100, 100), np.float32)], None, 0.5, 1.0, ())


@pytest.mark.parametrize("cfg,scale", [("5", 0.05), ("5t", 0.2)])
def test_block_configuration_scaled(ctx, cfg, scale):
    ws = W.config(cfg, scale=scale)
    check(ctx, "block", ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse)


# ---------------------------------------------------------------- full sizes
@pytest.mark.parametrize("cfg", ["4", "5"])
def test_full_size_configurations(ctx, cfg):
    ws = W.config(cfg)
    got, res, _ = check(ctx, ws.op, ws.w, ws.lam, ws.sparsity, ws.mu, ws.fuse)
    assert res.n_units == {"4": 62367776, "5": 8490000}[cfg]


# ---------------------------------------------------------------- arguments
def test_argument_errors_leave_buffers_untouched(ctx):
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ws = W.random_set([(64,), (8, 8)], seed=0)
    ds = DeviceSet(ws.w, ws.lam)
    ds.poison_outputs()
    bad = [lambda: ds.run(ctx, "prune", 1.5, 1e-3), lambda: ds.run(ctx, "prune", float("nan"), 1e-3),
           lambda: ds.run(ctx, "prune", 0.5, 0.0), lambda: ds.run(ctx, "prune", 0.5, float("inf")),
           lambda: ds.run(ctx, "prune", 0.5, -1.0), lambda: ds.run(ctx, "prune", 0.5, 1e-3, fuse=128), lambda: ds.run(ctx, "prune", 0.5, 1e-3, fuse=1 | 16),
           lambda: ds.run(ctx, "lagrange", 0.0, 1e-3, fuse=())]
    for f in bad:
        with pytest.raises(cstep.CondensaError) as e:
            f()
        assert e.value.code == cstep.ERR_INVALID_ARG
    with pytest.raises(cstep.CondensaError) as e:
        ds.run(ctx, "block", 0.5, 1e-3, block=(5000, 4))
    assert e.value.code == cstep.ERR_UNSUPPORTED
    with pytest.raises(cstep.CondensaError) as e:
        ds.run(ctx, "block", 0.5, 1e-3, block=(0, 4))
    assert e.value.code == cstep.ERR_INVALID_ARG
    with pytest.raises(cstep.CondensaError) as e:
        ctx.cstep_quantize(ds.table, ds.T, 1e-3, dtype=7)
    assert e.value.code == cstep.ERR_UNSUPPORTED
    # aliasing: theta on top of w; the same lambda twice
    tab = cstep.tensor_table(ds.w, ds.lam, ds.w, shapes=ds.shapes)
    with pytest.raises(cstep.CondensaError):
        ctx.cstep_prune(tab, ds.T, 0.5, 1e-3, ("lambda",))
    tab = cstep.tensor_table([ds.w[0], ds.w[0]], [ds.lam[0], ds.lam[0]], [ds.theta[0], ds.theta[1]],
                             shapes=[(64,), (64,)])
    with pytest.raises(cstep.CondensaError):
        ctx.cstep_prune(tab, 2, 0.5, 1e-3, ("lambda",))
    tab = cstep.tensor_table(ds.w, ds.lam, ds.theta, shapes=[(63,), (8, 8)])
    tab[0].numel = 64
    with pytest.raises(cstep.CondensaError):
        ctx.cstep_prune(tab, ds.T, 0.5, 1e-3)
    out = ds.fetch()
    assert all(np.isnan(t).all() for t in out["theta"]) and all((m == 7).all() for m in out["mask"])


def test_host_entry_point_matches_device_entry_point(ctx):
    from paper_1911_02497_b200 import cstep
    ws = W.config(2, scale=0.2)
    exp = oracle.cstep_prune(ws.w, ws.lam, 0.95, ws.mu, ("fp16", "lambda", "penalty"))
    w = [np.ascontiguousarray(a) for a in ws.w]
    lam = [a.copy() for a in ws.lam]
    theta = [np.empty_like(a) for a in w]
    mask = [np.empty(a.shape, np.uint8) for a in w]
    grad = [np.empty_like(a) for a in w]
    th = [np.empty(a.shape, np.uint16) for a in w]
    tab = cstep.tensor_table(w, lam, theta, mask, grad, th)
    ctx.cstep_host(cstep.OP_PRUNE, tab, len(w), 0.95, ws.mu, fuse=("fp16", "lambda", "penalty"))
    for t in range(len(w)):
        assert np.array_equal(mask[t], exp.mask[t]) and np.array_equal(th[t], exp.theta_h[t])
        assert np.array_equal(bits(theta[t]), bits(exp.theta[t]))
        assert np.array_equal(bits(lam[t]), bits(exp.lam[t]))
        assert np.array_equal(bits(grad[t]), bits(exp.grad[t]))


def test_deterministic_across_runs(ctx):
    ws = W.config(1, scale=0.5)
    first, _ = run_gpu(ctx, "prune", ws.w, ws.lam, 0.9, ws.mu, ws.fuse)
    for _ in range(5):
        again, _ = run_gpu(ctx, "prune", ws.w, ws.lam, 0.9, ws.mu, ws.fuse)
        for key in ("theta", "mask", "lam", "theta_h"):
            for a, b in zip(first[key], again[key]):
                assert np.array_equal(a.view(np.uint8), b.view(np.uint8))


def test_workspace_query_sizes_a_context_that_never_allocates():
    """condensa_workspace_bytes() tells how much condensa_create() must reserve: a context made
    with that figure runs the call without touching the device allocator."""
    import torch
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ws = W.config("5", scale=0.2)
    ds = DeviceSet(ws.w, ws.lam)
    need = cstep.workspace_bytes(cstep.OP_BLOCK, ds.table, ds.T, ("lambda",))
    assert need > 0
    # the first launch of a kernel in a process makes the CUDA runtime load its code, which takes
    # device memory of its own: a throw-away context runs the same call first
    c0 = cstep.Context(0)
    ds.run(c0, "block", ws.sparsity, ws.mu, ("lambda",))
    torch.cuda.synchronize()
    c0.close()
    ds.reset_lambda()
    c = cstep.Context(0, need)
    try:
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info(0)
        ds.run(c, "block", ws.sparsity, ws.mu, ("lambda",))
        assert c.get_result().sampled == 1
        free1, _ = torch.cuda.mem_get_info(0)
        assert free1 == free0
    finally:
        c.close()
    with pytest.raises(cstep.CondensaError):
        cstep.workspace_bytes(99, ds.table, ds.T)
    # the same for 5 x 5 blocks, which take a single-pass kernel of their own (larger journal)
    spec = cstep.StructureSpec(cstep.SPEC_BLOCKS, 0, cstep.CRITERIA["l2"], 2, (5, 5, 1, 1))
    need5 = cstep.workspace_bytes(cstep.OP_BLOCK, ds.table, ds.T, ("lambda",), C.byref(spec))
    assert need5 >= need
    c0 = cstep.Context(0)
    ds.reset_lambda()
    ds.run(c0, "block", ws.sparsity, ws.mu, ("lambda",), (5, 5))
    torch.cuda.synchronize()
    c0.close()
    ds.reset_lambda()
    c = cstep.Context(0, need5)
    try:
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info(0)
        ds.run(c, "block", ws.sparsity, ws.mu, ("lambda",), (5, 5))
        assert c.get_result().sampled == 1
        free1, _ = torch.cuda.mem_get_info(0)
        assert free1 == free0
    finally:
        c.close()


def test_register_resident_route_of_short_lists(ctx):
    """Lists of at most one work item per resident CTA are pruned in one launch out of registers:
    many small tensors with unaligned heads, every quantisation type, tie groups that are kept
    whole, cut in the middle (index levels) and spread over tensors, k = 0 and k = S."""
    shapes = [(4097,), (33, 17), (5, 3, 3, 3), (1,), (100003,), (64, 1500), (7,)]
    ws = W.random_set(shapes, seed=60, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    for s_ in (0.0, 0.37, 0.9, 1.0, 1e-6, 1 - 1e-6):
        got, res, _ = check(ctx, "prune", ws.w, ws.lam, s_, ws.mu, ("lambda", "penalty"))
        assert res.sampled == 0 and res.n_candidates == 0
    for q in ("fp16", "bf16", "e4m3", "e5m2"):
        check(ctx, "prune", ws.w, ws.lam, 0.8, ws.mu, (q, "lambda"), elem_offset=1)
    check(ctx, "prune", ws.w, [None] * len(shapes), 0.5, 1.0, (), skew=1)
    # ties: integers, so that many units share the threshold key
    ints = [np.round(a * 60).astype(np.float32) for a in ws.w]
    for s_ in (0.3, 0.5, 0.77):
        got, res, _ = check(ctx, "prune", ints, None, s_, 1.0, ("lambda",))
        assert res.n_tie > 1
    const = [np.full(n, v, np.float32) for n, v in ((5000, 0.5), (70001, -0.5), (3, 0.5))]
    for s_ in (0.1, 0.5, 0.999):
        got, res, _ = check(ctx, "prune", const, None, s_, 1.0, ())
        assert res.n_tie == 75004
    # the largest list the route takes on this device, and the first one it does not take
    import torch
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for n_items, route in ((2 * sms, 0), (2 * sms + 1, None)):
        n = 4096 * n_items
        w = W.draw(n, "normal", 0.05, 61, 0, 0)
        got, res, _ = check(ctx, "prune", [w], [np.zeros_like(w)], 0.9, 1e-3, ("fp16", "lambda"))
        if route is not None:
            assert res.sampled == route and res.n_candidates == 0
