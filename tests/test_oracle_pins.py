"""Pins for the CPU oracle: each test checks it against something other than
itself - the argmin definition by brute force, closed forms, numpy library
routines, hand-computed IEEE binary16 values."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from paper_1911_02497_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


def keys_of(u):
    return (bits(u) & np.uint32(0x7FFFFFFF)).astype(np.uint64)


def brute_keep(keys, k):
    """Definition of the ranking, O(n^2): unit i is kept iff fewer than k units
    precede it (larger key, or equal key and lower index)."""
    keys = np.asarray(keys).reshape(-1)
    n = keys.size
    idx = np.arange(n)
    keep = np.zeros(n, np.uint8)
    for i in range(n):
        rank = int((keys > keys[i]).sum() + ((keys == keys[i]) & (idx < i)).sum())
        keep[i] = rank < k
    return keep


def flat(arrs):
    return np.concatenate([np.asarray(a).reshape(-1) for a in arrs])


def test_denormals_and_struct_layout():
    assert oracle.lib().orc_denormals_ok() == 1


# ---------------------------------------------------------------- rounding of Z
def test_round_count_is_half_up_in_double():
    assert oracle.round_count(0.9, 1048576) == 943718
    assert oracle.round_count(0.95, 851504) == 808929
    assert oracle.round_count(0.98, 62367776) == 61120420
    assert oracle.round_count(0.8, 5504) == 4403
    assert oracle.round_count(0.9, 8490000) == 7641000
    assert oracle.round_count(0.5, 3) == 2          # 1.5 rounds up, not to even
    assert oracle.round_count(0.5, 5) == 3
    assert oracle.round_count(0.0, 7) == 0 and oracle.round_count(1.0, 7) == 7
    assert oracle.round_count(0.07, 7) == 0 and oracle.round_count(0.08, 7) == 1


# ---------------------------------------------------------------- u = w - lambda/mu
def test_form_u_hand_values_and_fp64_bound():
    w = np.array([1.0, 0.5, -2.0, 3.0], np.float32)
    lam = np.array([0.25, -0.125, 0.0, 1.5], np.float32)
    u = oracle.form_u(w, lam, 0.5)
    assert u.tolist() == [0.5, 0.75, -2.0, 0.0]
    assert np.array_equal(bits(oracle.form_u(w, None, 0.5)), bits(w))
    assert np.array_equal(bits(oracle.form_u(w, np.zeros(4, np.float32), 1e-3)), bits(w))
    rng = np.random.default_rng(1)
    w = rng.standard_normal(4096).astype(np.float32)
    lam = (rng.standard_normal(4096) * 1e-2).astype(np.float32)
    mu = np.float32(1e-3)
    u = oracle.form_u(w, lam, float(mu))
    # each step is one correctly rounded fp32 operation
    q = (lam.astype(np.float64) / np.float64(mu)).astype(np.float32)
    ref = (w.astype(np.float64) - q.astype(np.float64)).astype(np.float32)
    assert np.array_equal(bits(u), bits(ref))


# ---------------------------------------------------------------- unstructured
@pytest.mark.parametrize("n,s", [(1, 0.0), (1, 1.0), (7, 0.5), (64, 0.9), (257, 0.33),
                                 (2048, 0.95), (1000, 1.0 / 1000), (1000, 1 - 1.0 / 1000)])
def test_prune_matches_bruteforce_rank(n, s):
    ws = W.random_set([(n,)], seed=n, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    out = oracle.cstep_prune(ws.w, ws.lam, s, ws.mu, ("lambda",))
    u = oracle.form_u(ws.w[0], ws.lam[0], ws.mu)
    z = int(math.floor(s * n + 0.5))
    keep = brute_keep(keys_of(u), n - z)
    assert np.array_equal(out.mask[0].reshape(-1), keep)
    assert int((out.mask[0] == 0).sum()) == z == out.result.n_zero
    # kept entries equal u bit for bit, pruned entries are +0
    tb = bits(out.theta[0]).reshape(-1)
    assert np.array_equal(tb[keep == 1], bits(u).reshape(-1)[keep == 1])
    assert np.all(tb[keep == 0] == 0)


def test_prune_is_the_argmin_over_all_supports():
    """C(w) = argmin ||u - theta||^2 over theta with at most k non-zeros:
    enumerate every support of size k on tiny inputs."""
    rng = np.random.default_rng(7)
    for n, k in [(6, 2), (9, 4), (12, 3), (10, 9), (8, 0)]:
        w = rng.standard_normal(n).astype(np.float32)
        s = (n - k) / n
        out = oracle.cstep_prune([w], [None], s, 1.0, ())
        assert out.result.n_keep == k
        got = float(((w.astype(np.float64) - out.theta[0].astype(np.float64)) ** 2).sum())
        best = min(float((np.delete(w.astype(np.float64), list(sup)) ** 2).sum())
                   for sup in itertools.combinations(range(n), k))
        assert got == pytest.approx(best, rel=1e-12, abs=1e-300)


def test_prune_threshold_against_partition_and_invariants():
    ws = W.config(2, scale=0.25)
    out = oracle.cstep_prune(ws.w, ws.lam, 0.95, ws.mu, ("lambda",))
    u = flat([oracle.form_u(w, l, ws.mu) for w, l in zip(ws.w, ws.lam)])
    key = keys_of(u)
    n = key.size
    k = out.result.n_keep
    tau = np.partition(key, n - k)[n - k]          # k-th largest via a library selection
    assert int(tau) == out.result.tau_key
    assert int((key > tau).sum()) == out.result.n_gt < k <= int((key >= tau).sum())
    assert out.result.n_tie == int((key == tau).sum())
    m = flat(out.mask)
    assert int(m.sum()) == k
    assert np.all(m[key > tau] == 1) and np.all(m[key < tau] == 0)
    assert out.result.tau_id == int(np.flatnonzero((key == tau) & (m == 1)).max())


def test_prune_tie_rule_lowest_index_first():
    c = np.full(10, 0.5, np.float32)
    out = oracle.cstep_prune([c], [None], 0.7, 1.0, ())
    assert out.mask[0].tolist() == [1, 1, 1, 0, 0, 0, 0, 0, 0, 0]
    assert (out.result.n_gt, out.result.n_tie, out.result.n_tie_kept, out.result.tau_id) == (0, 10, 3, 2)
    # +x and -x tie; zeros and negative zeros tie with key 0
    w = np.array([-1.0, 1.0, 0.0, -0.0, 1.0, -1.0], np.float32)
    out = oracle.cstep_prune([w], [None], 0.5, 1.0, ())
    assert out.mask[0].tolist() == [1, 1, 0, 0, 1, 0]
    # ties straddling a tensor boundary: the global index decides
    a = np.array([2.0, 1.0], np.float32)
    b = np.array([1.0, 1.0, 3.0], np.float32)
    out = oracle.cstep_prune([a, b], [None, None], 0.4, 1.0, ())
    assert out.mask[0].tolist() == [1, 1] and out.mask[1].tolist() == [0, 0, 1]
    # all zero
    z = np.zeros(5, np.float32)
    out = oracle.cstep_prune([z], [None], 0.6, 1.0, ())
    assert out.mask[0].tolist() == [1, 1, 0, 0, 0] and np.all(bits(out.theta[0]) == 0)


def test_prune_k_zero_and_keep_all():
    w = np.array([3.0, -1.0, 2.0], np.float32)
    out = oracle.cstep_prune([w], [None], 1.0, 1.0, ())
    assert out.mask[0].sum() == 0 and out.result.tau_key == 0x7F800000 and out.result.tau_id == -1
    out = oracle.cstep_prune([w], [None], 0.0, 1.0, ())
    assert out.mask[0].sum() == 3 and out.result.tau_key == 0x3F800000
    assert np.array_equal(bits(out.theta[0]), bits(w))


def test_prune_nan_and_inf_order():
    w = np.array([1.0, np.inf, np.nan, -np.inf, 0.5], np.float32)
    out = oracle.cstep_prune([w], [None], 0.6, 1.0, ())
    assert out.mask[0].tolist() == [0, 1, 1, 0, 0]   # NaN key above inf; lower index inf first


def test_prune_idempotent():
    ws = W.random_set([(33, 17), (500,)], seed=5, kind="normal", scale=0.1)
    a = oracle.cstep_prune(ws.w, [None, None], 0.8, 1.0, ())
    b = oracle.cstep_prune(a.theta, [None, None], 0.8, 1.0, ())
    for x, y, mx, my in zip(a.theta, b.theta, a.mask, b.mask):
        assert np.array_equal(bits(x), bits(y))
        assert np.array_equal(mx, my)              # tau > 0 here, so the masks agree too


# ---------------------------------------------------------------- structures
def test_block_norm_closed_forms():
    c = np.float32(0.375)
    w = np.full((6, 8), c, np.float32)             # rows 4..5 form ragged blocks of 2 x 4
    nu = oracle.structure_norms([w], [None], 1.0, "block")
    assert nu.tolist() == [16 * float(c) ** 2] * 2 + [8 * float(c) ** 2] * 2
    w = np.zeros((4, 8), np.float32); w[2, 5] = 3.0
    assert oracle.structure_norms([w], [None], 1.0, "block").tolist() == [0.0, 9.0]
    rng = np.random.default_rng(3)
    w = rng.integers(-4096, 4097, size=(9, 10)).astype(np.float32)   # exact in any order
    nu = oracle.structure_norms([w], [None], 1.0, "block")
    ref = []
    for br in range(3):
        for bc in range(3):
            ref.append(float((w[4 * br:4 * br + 4, 4 * bc:4 * bc + 4].astype(np.float64) ** 2).sum()))
    assert nu.tolist() == ref
    # general block shape, against long-double accumulation
    w = rng.standard_normal((11, 13)).astype(np.float32)
    nu = oracle.structure_norms([w], [None], 1.0, "block", (5, 5))
    k = 0
    for br in range(3):
        for bc in range(3):
            blk = w[5 * br:5 * br + 5, 5 * bc:5 * bc + 5].astype(np.longdouble)
            assert nu[k] == pytest.approx(float((blk * blk).sum()), rel=1e-14)
            k += 1
    assert k == nu.size


def test_filter_norm_closed_forms_and_passthrough():
    w = np.zeros((3, 2, 3, 3), np.float32)
    w[0] = 0.5; w[1, 1, 2, 0] = -2.0
    fc = np.ones((4, 5), np.float32)
    nu = oracle.structure_norms([w, fc], [None, None], 1.0, "filter")
    assert nu.tolist() == [18 * 0.25, 4.0, 0.0]
    rng = np.random.default_rng(11)
    w = rng.standard_normal((5, 7, 3, 3)).astype(np.float32)
    lam = (rng.standard_normal(w.shape) * 0.01).astype(np.float32)
    nu = oracle.structure_norms([w], [lam], 0.01, "filter")
    u = oracle.form_u(w, lam, 0.01).astype(np.longdouble).reshape(5, -1)
    assert np.allclose(nu, (u * u).sum(1).astype(np.float64), rtol=1e-14, atol=0)


@pytest.mark.parametrize("kind", ["filter", "block"])
def test_structured_kept_set_bruteforce(kind):
    if kind == "filter":
        shapes, s = [(7, 3, 3, 3), (10, 12), (9, 7, 1, 1)], 0.6
    else:
        shapes, s = [(10, 14), (5,), (7, 9)], 0.55
    ws = W.random_set(shapes, seed=21, kind="normal", scale=0.2, lam_sigma=1e-2, mu=1e-2)
    fn = oracle.cstep_filter if kind == "filter" else oracle.cstep_block
    out = fn(ws.w, ws.lam, s, ws.mu, fuse=("lambda",))
    nu = oracle.structure_norms(ws.w, ws.lam, ws.mu, kind)
    S = nu.size
    z = int(math.floor(s * S + 0.5))
    keep_s = brute_keep(nu.view(np.uint64), S - z)
    assert out.result.n_units == S and out.result.n_zero == z
    sid = 0
    for t, shp in enumerate(shapes):
        u = oracle.form_u(ws.w[t], ws.lam[t], ws.mu)
        m = out.mask[t]
        ranked = (len(shp) == 4) if kind == "filter" else (len(shp) == 2)
        if not ranked:
            assert m.all() and np.array_equal(bits(out.theta[t]), bits(u))
            continue
        if kind == "filter":
            exp = np.repeat(keep_s[sid:sid + shp[0]], int(np.prod(shp[1:]))).reshape(shp)
            sid += shp[0]
        else:
            nbr, nbc = -(-shp[0] // 4), -(-shp[1] // 4)
            grid = keep_s[sid:sid + nbr * nbc].reshape(nbr, nbc)
            exp = np.kron(grid, np.ones((4, 4), np.uint8))[:shp[0], :shp[1]]
            sid += nbr * nbc
        assert np.array_equal(m, exp)
        assert np.array_equal(bits(out.theta[t]), np.where(exp == 1, bits(u), 0))
    assert sid == S
    assert out.result.tau_norm == pytest.approx(math.sqrt(nu[out.result.tau_id]), rel=1e-6)


def test_structured_argmin_over_all_supports():
    rng = np.random.default_rng(5)
    w = rng.standard_normal((8, 12)).astype(np.float32)       # 2 x 3 = 6 blocks
    for k in (0, 1, 3, 5, 6):
        out = oracle.cstep_block([w], [None], (6 - k) / 6, 1.0)
        got = float(((w.astype(np.float64) - out.theta[0]) ** 2).sum())
        nu = [float((w[4 * r:4 * r + 4, 4 * c:4 * c + 4].astype(np.float64) ** 2).sum())
              for r in range(2) for c in range(3)]
        best = min(sum(nu) - sum(nu[i] for i in sup) for sup in itertools.combinations(range(6), k))
        assert got == pytest.approx(best, rel=1e-12)
    f = rng.standard_normal((5, 2, 3, 3)).astype(np.float32)
    out = oracle.cstep_filter([f], [None], 0.6, 1.0)
    nu = (f.astype(np.float64).reshape(5, -1) ** 2).sum(1)
    assert sorted(np.flatnonzero(out.mask[0].reshape(5, -1)[:, 0]).tolist()) == sorted(
        np.argsort(-nu)[:2].tolist())


def test_structured_ties_use_structure_index():
    blk = np.arange(16, dtype=np.float32).reshape(4, 4)
    w = np.tile(blk, (2, 3))                                   # six identical blocks
    out = oracle.cstep_block([w], [None], 0.5, 1.0)
    grid = out.mask[0][::4, ::4]
    assert grid.tolist() == [[1, 1, 1], [0, 0, 0]]
    assert out.result.n_tie == 6 and out.result.n_tie_kept == 3 and out.result.tau_id == 2


@pytest.mark.parametrize("block", [(5, 5), (3, 2), (1, 8), (8, 1), (2, 7)])
def test_general_block_shapes_kept_set_mask_and_theta_bruteforce(block):
    """BlockPrune with any block shape (Table 1; the LSTM run of the Evaluation uses
    bs = 5): norms from numpy slices, kept set from the O(n^2) rank definition, the
    element mask by np.kron of the block grid - non-square and ragged on purpose, so
    that exchanging block height and width anywhere in the oracle fails here."""
    bh, bw = block
    shapes, s = [(11, 13), (6,), (33, 28)], 0.55
    ws = W.random_set(shapes, seed=31, kind="normal", scale=0.2, lam_sigma=1e-2, mu=1e-2)
    out = oracle.cstep_block(ws.w, ws.lam, s, ws.mu, block, fuse=("lambda",))
    nu_ref = []
    for t, shp in enumerate(shapes):
        if len(shp) != 2:
            continue
        u = oracle.form_u(ws.w[t], ws.lam[t], ws.mu).astype(np.float64)
        for br in range(-(-shp[0] // bh)):
            for bc in range(-(-shp[1] // bw)):
                blk = u[bh * br:bh * br + bh, bw * bc:bw * bc + bw]
                acc = 0.0
                for x in blk.reshape(-1):          # row by row inside the block
                    acc = acc + x * x
                nu_ref.append(acc)
    nu_ref = np.array(nu_ref, np.float64)
    nu = oracle.structure_norms(ws.w, ws.lam, ws.mu, "block", block)
    assert np.array_equal(nu.view(np.uint64), nu_ref.view(np.uint64))
    S = nu_ref.size
    z = int(math.floor(s * S + 0.5))
    keep_s = brute_keep(nu_ref.view(np.uint64), S - z)
    assert out.result.n_units == S and out.result.n_zero == z and int(keep_s.sum()) == S - z
    sid = 0
    for t, shp in enumerate(shapes):
        u = oracle.form_u(ws.w[t], ws.lam[t], ws.mu)
        if len(shp) != 2:
            assert out.mask[t].all() and np.array_equal(bits(out.theta[t]), bits(u))
            continue
        nbr, nbc = -(-shp[0] // bh), -(-shp[1] // bw)
        grid = keep_s[sid:sid + nbr * nbc].reshape(nbr, nbc)
        exp = np.kron(grid, np.ones((bh, bw), np.uint8))[:shp[0], :shp[1]]
        sid += nbr * nbc
        assert np.array_equal(out.mask[t], exp)
        assert np.array_equal(bits(out.theta[t]), np.where(exp == 1, bits(u), 0))
        # multiplier update on top of that theta: lambda' = lambda - mu (w - theta)
        th = np.where(exp == 1, u, np.float32(0))
        lam_ref = ws.lam[t] - np.float32(ws.mu) * (ws.w[t] - th)
        assert np.array_equal(bits(out.lam[t]), bits(lam_ref.astype(np.float32)))
    assert sid == S
    kept_ids = np.flatnonzero(keep_s)
    weakest = kept_ids[np.lexsort((-kept_ids, nu_ref[kept_ids]))[0]]
    assert out.result.tau_id == weakest


def test_general_block_ties_use_block_index():
    blk = np.arange(6, dtype=np.float32).reshape(3, 2) + 1
    w = np.tile(blk, (2, 4))                                   # 2 x 4 identical 3x2 blocks
    out = oracle.cstep_block([w], [None], 0.5, 1.0, (3, 2))
    assert out.mask[0][::3, ::2].tolist() == [[1, 1, 1, 1], [0, 0, 0, 0]]
    assert out.result.n_tie == 8 and out.result.n_tie_kept == 4 and out.result.tau_id == 3
    out = oracle.cstep_block([w.T.copy()], [None], 0.25, 1.0, (2, 3))     # 4 x 2 blocks of 2x3
    assert out.mask[0][::2, ::3].tolist() == [[1, 1], [1, 1], [1, 1], [0, 0]]


def test_filter_and_neuron_ties_use_structure_index():
    """Bit-identical filters tie: the lower global structure id is kept, within a
    tensor and across tensors, for FilterPrune and for the mixed StructurePrune list."""
    rng = np.random.default_rng(17)
    f = rng.standard_normal((1, 3, 3, 3)).astype(np.float32)
    a = np.repeat(f, 4, axis=0)                                # four identical filters
    b = np.repeat(f, 3, axis=0)
    out = oracle.cstep_filter([a, b], [None, None], 3 / 7, 1.0)   # Z = 3 of 7, all tied
    assert out.result.n_tie == 7 and out.result.n_tie_kept == 4 and out.result.tau_id == 3
    assert out.mask[0].all() and not out.mask[1].any()
    strong = (2 * f).astype(np.float32)
    c = np.concatenate([f, strong, f, f], axis=0)              # ids 0..3, id 1 is the strongest
    out = oracle.cstep_filter([c], [None], 0.5, 1.0)           # keep 2: id 1, then the lowest tied id 0
    assert out.mask[0].reshape(4, -1)[:, 0].tolist() == [1, 1, 0, 0]
    assert out.result.n_gt == 1 and out.result.n_tie == 3 and out.result.n_tie_kept == 1 and out.result.tau_id == 0
    # rows of a matrix that equal a filter, ranked together with it
    row = f.reshape(1, 27)
    m = np.concatenate([row, row], axis=0)
    out = oracle.cstep_structure([m, a], [None, None], 0.5, 1.0, ("filter", "neuron"))   # 6 tied, keep ids 0..2
    assert out.mask[0].all() and out.mask[1].reshape(4, -1)[:, 0].tolist() == [1, 0, 0, 0]
    assert out.result.tau_id == 2 and out.result.n_tie == 6


# ---------------------------------------------------------------- binary16
def _golden_f16():
    rows = []
    with open(os.path.join(GOLD, "binary16_hand_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                a, b = line.split()
                rows.append((int(a, 16), int(b, 16)))
    return rows


def test_f16_hand_values():
    rows = _golden_f16()
    assert len(rows) >= 20
    for fb, hb in rows:
        assert int(oracle.lib().orc_f32_to_f16(fb)) == hb, hex(fb)


def test_f16_roundtrip_and_midpoints():
    allh = np.arange(65536, dtype=np.uint16)
    wide = allh.view(np.float16).astype(np.float32)           # numpy widening: exact
    mine = oracle.f16_bits_to_f32(allh)
    nan = np.isnan(wide)
    assert np.array_equal(bits(mine)[~nan], bits(wide)[~nan])
    assert np.all(np.isnan(mine[nan]))
    back = oracle.f32_to_f16_bits(wide)
    assert np.array_equal(back[~nan], allh[~nan])
    # midpoint of two adjacent finite positive halves goes to the even one
    h = np.arange(0, 0x7BFF, dtype=np.uint16)
    a = h.view(np.float16).astype(np.float64)
    b = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((a + b) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (a + b) / 2)     # midpoints are exact in fp32
    got = oracle.f32_to_f16_bits(mid)
    even = np.where(h % 2 == 0, h, h + 1).astype(np.uint16)
    assert np.array_equal(got, even)
    got_neg = oracle.f32_to_f16_bits(-mid)
    assert np.array_equal(got_neg, even | np.uint16(0x8000))


def test_f16_against_numpy_conversion():
    """numpy's float32 -> float16 cast is an independent IEEE implementation."""
    rng = np.random.default_rng(0)
    pats = [rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)]
    # every exponent with the rounding-critical low mantissa patterns
    e = np.arange(256, dtype=np.uint32)[:, None, None] << 23
    hi = (rng.integers(0, 1 << 10, size=(1, 64, 1), dtype=np.uint64).astype(np.uint32)) << 13
    lo = np.array([0, 1, 0x0FFF, 0x1000, 0x1001, 0x1FFF], np.uint32)[None, None, :]
    crit = (e | hi | lo).reshape(-1)
    pats += [crit, crit | np.uint32(0x80000000)]
    # the whole subnormal-half range boundary region, densely
    pats.append(np.arange(0x33000000 - 4096, 0x33000000 + 4096, dtype=np.uint32))
    pats.append(np.arange(0x38800000 - 70000, 0x38800000 + 70000, dtype=np.uint32))
    pats.append(np.arange(0x477FE000 - 9000, 0x477FE000 + 9000, dtype=np.uint32))
    p = np.concatenate(pats)
    x = p.view(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = oracle.f32_to_f16_bits(p)
    nan = np.isnan(x)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all((got[nan] & 0x7FFF) == 0x7E00)
    assert np.array_equal(got[nan] >> 15, (p[nan] >> 31).astype(np.uint16))


def test_quantize_scheme_and_pq_order():
    ws = W.config(1, scale=1 / 64)
    out = oracle.cstep_prune(ws.w, ws.lam, 0.9, ws.mu, ("fp16", "lambda"))
    u = oracle.form_u(ws.w[0], ws.lam[0], ws.mu)
    plain = oracle.cstep_prune(ws.w, ws.lam, 0.9, ws.mu, ())
    assert np.array_equal(out.mask[0], plain.mask[0])          # ranking uses un-quantised u
    with np.errstate(over="ignore"):
        q = u.astype(np.float16)
    exp = np.where(plain.mask[0] == 1, q.astype(np.float32), np.float32(0))
    assert np.array_equal(bits(out.theta[0]), bits(exp))
    assert np.array_equal(out.theta_h[0], np.where(plain.mask[0] == 1, q.view(np.uint16), 0))
    qo = oracle.cstep_quantize(ws.w, ws.lam, ws.mu, ())
    assert np.array_equal(bits(qo.theta[0]), bits(q.astype(np.float32))) and qo.mask[0].all()
    # footprint closed form: fp32 bytes over fp16 bytes of the non-zeros = 2 / (1 - s)
    nnz = int((out.theta[0] != 0).sum())
    ratio = 4 * ws.numel / (2 * nnz)
    assert ratio == pytest.approx(2 / (1 - 0.9), rel=2e-3)


# ---------------------------------------------------------------- multipliers
def test_lagrange_hand_case_and_fixed_point():
    w = np.array([1.0], np.float32); th = np.array([0.25], np.float32)
    lam = np.array([0.125], np.float32)
    out = oracle.lagrange_update([w], [th], [lam], 0.5, ("lambda", "penalty"))
    assert out.lam[0].tolist() == [-0.25] and out.grad[0].tolist() == [0.625]
    out = oracle.lagrange_update([w], [th], [lam], 0.5, ("penalty",))
    assert out.lam[0].tolist() == [0.125] and out.grad[0].tolist() == [0.25]
    rng = np.random.default_rng(2)
    w = rng.standard_normal(1000).astype(np.float32)
    lam = rng.standard_normal(1000).astype(np.float32)
    out = oracle.lagrange_update([w], [w.copy()], [lam], 1e-3, ("lambda", "penalty"))
    assert np.array_equal(bits(out.lam[0]), bits(lam))          # w == theta: lambda unchanged
    assert np.array_equal(bits(out.grad[0]), bits(np.float32(0) - lam))
    out = oracle.lagrange_update([w], [w.copy()], [np.zeros_like(w)], 1e-3, ("lambda",))
    assert np.all(bits(out.lam[0]) == 0)                        # lambda stays zero


def test_lagrange_matches_fp64_recomputation():
    ws = W.random_set([(4096,)], seed=9, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
    out = oracle.cstep_prune(ws.w, ws.lam, 0.7, ws.mu, ("lambda", "penalty"))
    w, lam, th = (a[0].astype(np.float64) for a in (ws.w, ws.lam, out.theta))
    mu = np.float64(np.float32(ws.mu))
    d = (w - th).astype(np.float32)
    p = (mu * d.astype(np.float64)).astype(np.float32)
    l2 = (lam - p.astype(np.float64)).astype(np.float32)
    g = (p.astype(np.float64) - l2.astype(np.float64)).astype(np.float32)
    assert np.array_equal(bits(out.lam[0]), bits(l2))
    assert np.array_equal(bits(out.grad[0]), bits(g))
    exact = mu * (w - th) - (lam - mu * (w - th))
    assert np.allclose(out.grad[0], exact, rtol=1e-5, atol=1e-9)


def test_null_lambda_means_zero_and_no_update():
    w = np.array([0.5, -1.5, 2.0, 0.1], np.float32)
    out = oracle.cstep_prune([w], [None], 0.5, 0.25, ("lambda", "penalty"))
    assert out.mask[0].tolist() == [0, 1, 1, 0]
    assert out.lam[0].tolist() == [0, 0, 0, 0]
    assert out.grad[0].tolist() == [0.125, 0.0, 0.0, 0.025000000372529030]


# ---------------------------------------------------------------- generator
def test_generator_is_counter_based_and_has_the_right_moments():
    a = W.draw(100000, "normal", 0.05, seed=0, stream=0, tensor=0, threads=1)
    b = W.draw(100000, "normal", 0.05, seed=0, stream=0, tensor=0, threads=4)
    assert np.array_equal(a, b)
    part = W.draw(60000, "normal", 0.05, seed=0, stream=0, tensor=0)
    assert np.array_equal(part, a[:60000])
    assert abs(float(a.mean())) < 1e-3 and float(a.std()) == pytest.approx(0.05, rel=2e-2)
    u = W.draw(100000, "uniform", 0.1, seed=4, stream=0, tensor=3)
    assert -0.1 < u.min() < -0.099 and 0.099 < u.max() < 0.1
    assert float(u.std()) == pytest.approx(0.1 / math.sqrt(3), rel=2e-2)
    assert not np.array_equal(W.draw(64, "uniform", 0.1, 4, 0, 3), W.draw(64, "uniform", 0.1, 4, 1, 3))


def test_configuration_shapes():
    assert sum(int(np.prod(s)) for s in W.resnet56_shapes()) == 851504 and len(W.resnet56_shapes()) == 58
    assert sum(int(np.prod(s)) for s in W.vgg19_shapes()) == 20024000
    assert sum(s[0] for s in W.vgg19_shapes() if len(s) == 4) == 5504
    assert sum(int(np.prod(s)) for s in W.alexnet_shapes()) == 62367776
    assert sum(int(np.prod(s)) for s in W.lstm_lm_shapes()) == 135858000
    assert sum(int(np.prod(s)) for s in W.lstm_lm_shapes(tied=True)) == 85941000
    nb = sum(-(-s[0] // 4) * -(-s[1] // 4) for s in W.lstm_lm_shapes() if len(s) == 2)
    assert nb == 8490000


# ---------------------------------------------------------------- L-step update
def test_lstep_sgd_hand_case_and_torch_sgd():
    import torch
    # exactly representable numbers: mu (w - theta) - lambda = 0.5*(1-0.25) - 0.125 = 0.25; g = 1 + 0.25
    w, th, lam, g, b = (np.array([v], np.float32) for v in (1.0, 0.25, 0.125, 1.0, 2.0))
    wn, b1, _ = oracle.lstep_update([w], [th], [lam], [g], [b], None, 0.5, "sgd", lr=0.5, momentum=0.5)
    assert b1[0].tolist() == [2.25] and wn[0].tolist() == [-0.125]
    # against torch.optim.SGD fed with the same total gradient (an independent implementation)
    rng = np.random.default_rng(3)
    n = 5000
    w = rng.standard_normal(n).astype(np.float32); th = np.where(np.abs(w) > 1, w, 0).astype(np.float32)
    lam = (rng.standard_normal(n) * 0.01).astype(np.float32); g = rng.standard_normal(n).astype(np.float32)
    b = (rng.standard_normal(n) * 0.1).astype(np.float32)
    mu = 1e-2
    wn, b1, _ = oracle.lstep_update([w], [th], [lam], [g], [b], None, mu, "sgd", lr=0.1, momentum=0.9,
                                    weight_decay=1e-4)
    p = torch.nn.Parameter(torch.from_numpy(w.copy()))
    opt = torch.optim.SGD([p], lr=0.1, momentum=0.9, weight_decay=1e-4)
    opt.state[p]["momentum_buffer"] = torch.from_numpy(b.copy())
    p.grad = torch.from_numpy(g) + (np.float32(mu) * (torch.from_numpy(w) - torch.from_numpy(th)) - torch.from_numpy(lam))
    opt.step()
    assert np.allclose(wn[0], p.detach().numpy(), rtol=2e-6, atol=1e-7)
    assert np.allclose(b1[0], opt.state[p]["momentum_buffer"].numpy(), rtol=2e-6, atol=1e-7)
    # theta == w and lambda == 0: the penalty vanishes and the step is plain SGD
    wn2, _, _ = oracle.lstep_update([w], [w.copy()], [np.zeros_like(w)], [g], [np.zeros_like(w)], None, mu, "sgd",
                                    lr=0.1, momentum=0.9)
    assert np.array_equal(wn2[0].view(np.uint32), (w - np.float32(0.1) * g).astype(np.float32).view(np.uint32))


def test_lstep_adam_against_torch_adam():
    import torch
    rng = np.random.default_rng(4)
    n = 5000
    w = rng.standard_normal(n).astype(np.float32); th = np.where(np.abs(w) > 1, w, 0).astype(np.float32)
    lam = (rng.standard_normal(n) * 0.01).astype(np.float32); g = rng.standard_normal(n).astype(np.float32)
    m = (rng.standard_normal(n) * 0.1).astype(np.float32); v = (rng.random(n) * 0.1).astype(np.float32)
    mu, step = 1e-3, 7
    wn, m1, v1 = oracle.lstep_update([w], [th], [lam], [g], [m], [v], mu, "adam", lr=1e-4, beta1=0.9,
                                     beta2=0.999, eps=1e-8, step=step)
    p = torch.nn.Parameter(torch.from_numpy(w.copy()))
    # torch keeps its hyper-parameters in double: hand it the float values the oracle works with
    f32 = lambda x: float(np.float32(x))
    opt = torch.optim.Adam([p], lr=f32(1e-4), betas=(f32(0.9), f32(0.999)), eps=f32(1e-8))
    opt.state[p]["step"] = torch.tensor(float(step - 1))
    opt.state[p]["exp_avg"] = torch.from_numpy(m.copy())
    opt.state[p]["exp_avg_sq"] = torch.from_numpy(v.copy())
    p.grad = torch.from_numpy(g) + (np.float32(mu) * (torch.from_numpy(w) - torch.from_numpy(th)) - torch.from_numpy(lam))
    opt.step()
    # torch forms the first moment as m + (1-b1)(g - m): same value, other rounding (operands are O(1))
    assert np.allclose(m1[0], opt.state[p]["exp_avg"].numpy(), rtol=2e-6, atol=3e-7)
    assert np.allclose(v1[0], opt.state[p]["exp_avg_sq"].numpy(), rtol=2e-6, atol=3e-8)
    assert np.allclose(wn[0], p.detach().numpy(), rtol=1e-6, atol=1e-7)
    assert 1e-5 < np.abs(wn[0] - w).max() < 1e-3        # moved by about lr
    # closed form at step 1 from zero moments: m_hat = g, v_hat = g^2, so w moves by lr * sign(g) (eps aside)
    z = np.zeros(n, np.float32)
    wn, _, _ = oracle.lstep_update([w], [w.copy()], [z], [g], [z], [z], mu, "adam", lr=1e-3, step=1)
    big = np.abs(g) > 1e-3
    assert np.allclose((w - wn[0])[big], 1e-3 * np.sign(g[big]), rtol=1e-4)


# ---------------------------------------------------------------- neurons / structures
def test_neuron_and_structure_pruning():
    rng = np.random.default_rng(8)
    fc = rng.standard_normal((9, 7)).astype(np.float32)
    conv = (rng.standard_normal((4, 2, 3, 3)) * 0.5).astype(np.float32)
    bias = rng.standard_normal(5).astype(np.float32)
    # neurons only: rows of the 2-D tensor, everything else passes through
    nu = oracle.structure_norms([fc, conv, bias], [None] * 3, 1.0, "neuron")
    assert np.allclose(nu, (fc.astype(np.float64) ** 2).sum(1), rtol=1e-14) and nu.size == 9
    out = oracle.cstep_structure([fc, conv, bias], [None] * 3, 4 / 9, 1.0, ("neuron",))
    keep = brute_keep(nu.view(np.uint64), 5)
    assert np.array_equal(out.mask[0], np.repeat(keep, 7).reshape(9, 7))
    assert out.mask[1].all() and out.mask[2].all() and out.result.n_units == 9
    # both kinds in one ranking, numbered tensor by tensor (rows of fc first, then the filters)
    nu = oracle.structure_norms([fc, conv, bias], [None] * 3, 1.0, "structure")
    ref = np.concatenate([(fc.astype(np.float64) ** 2).sum(1), (conv.astype(np.float64).reshape(4, -1) ** 2).sum(1)])
    assert np.allclose(nu, ref, rtol=1e-14)
    out = oracle.cstep_structure([fc, conv, bias], [None] * 3, 0.5, 1.0, ("neuron", "filter"))
    keep = brute_keep(nu.view(np.uint64), 13 - 7)            # Z = floor(6.5 + 0.5) = 7
    assert np.array_equal(out.mask[0][:, 0], keep[:9]) and np.array_equal(out.mask[1][:, 0, 0, 0], keep[9:])
    assert int(out.mask[0][:, 0].sum() + out.mask[1][:, 0, 0, 0].sum()) == 6
    # the filter scheme is the same call with only the filter kind
    a = oracle.cstep_filter([fc, conv], [None, None], 0.5, 1.0)
    b = oracle.cstep_structure([fc, conv], [None, None], 0.5, 1.0, ("filter",))
    assert all(np.array_equal(x, y) for x, y in zip(a.mask, b.mask))


# ---------------------------------------------------------------- bfloat16
def test_bf16_hand_values_and_torch():
    import torch
    hand = {0x3F800000: 0x3F80,      # 1
            0x3F808000: 0x3F80,      # 1 + 2^-8 is the tie between 0x3F80 and 0x3F81: even
            0x3F818000: 0x3F82,      # 1 + 3*2^-8 ties up to the even 0x3F82
            0x3F808001: 0x3F81,      # just above the tie
            0x7F7F8000: 0x7F80,      # the tie above the largest bfloat16 goes to infinity
            0x7F7F7FFF: 0x7F7F,      # just below it stays finite
            0x80000000: 0x8000, 0x00000001: 0x0000, 0x00008000: 0x0000, 0x00008001: 0x0001,
            0x00018000: 0x0002,      # subnormal tie to even
            0x7F800000: 0x7F80, 0xFF800000: 0xFF80, 0x7FC00000: 0x7FC0, 0xFF800001: 0xFFC0,
            0x3DCCCCCD: 0x3DCD}      # 0.1f rounds up
    for fb, hb in hand.items():
        assert int(oracle.lib().orc_f32_to_bf16(fb)) == hb, hex(fb)
    rng = np.random.default_rng(5)
    pats = [rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)]
    hi = np.arange(0, 1 << 16, dtype=np.uint32)[:, None] << 16           # every bfloat16 with the critical tails
    lo = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF], np.uint32)[None, :]
    pats.append((hi | lo).reshape(-1))
    p = np.concatenate(pats)
    got = oracle.f32_to_bf16_bits(p)
    ref = torch.from_numpy(p.view(np.int32)).view(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(p.view(np.float32))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all((got[nan] & 0x7FFF) == 0x7FC0) and np.array_equal(got[nan] >> 15, (p[nan] >> 31).astype(np.uint16))
    # scheme level: prune then quantise to bfloat16
    ws = W.config(1, scale=1 / 64)
    out = oracle.cstep_prune(ws.w, ws.lam, 0.9, ws.mu, ("bf16", "lambda"))
    plain = oracle.cstep_prune(ws.w, ws.lam, 0.9, ws.mu, ())
    u = oracle.form_u(ws.w[0], ws.lam[0], ws.mu)
    q = torch.from_numpy(u).to(torch.bfloat16)
    exp = np.where(plain.mask[0] == 1, q.to(torch.float32).numpy(), np.float32(0))
    assert np.array_equal(out.mask[0], plain.mask[0]) and np.array_equal(bits(out.theta[0]), bits(exp))
    assert np.array_equal(out.theta_h[0], np.where(plain.mask[0] == 1, q.view(torch.int16).numpy().view(np.uint16), 0))


# ---------------------------------------------------------------- 8-bit floating point
def test_fp8_hand_values_roundtrip_midpoints_and_torch():
    """Quantize(dtype) with the two 8-bit formats: hand-worked values, every code widens and
    converts back to itself, every midpoint between neighbouring codes goes to the even one,
    and torch's independent cast agrees wherever the value is inside the format's range."""
    import torch
    rows = []
    with open(os.path.join(GOLD, "fp8_hand_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                fmt, a, b = line.split()
                rows.append((fmt, int(a, 16), int(b, 16)))
    assert len(rows) >= 30
    for fmt, fb, code in rows:
        assert int(oracle.lib().orc_f32_to_fp8(fb, oracle.FP8_FORMATS[fmt])) == code, (fmt, hex(fb))
    for fmt, tdt, top in (("e4m3", torch.float8_e4m3fn, 0x7E), ("e5m2", torch.float8_e5m2, 0x7B)):
        codes = np.array([c for c in range(256) if (c & 0x7F) <= top], np.uint8)        # the finite codes
        wide = oracle.fp8_bits_to_f32(codes, fmt)
        ref = torch.from_numpy(codes.copy()).view(tdt).to(torch.float32).numpy()        # torch's widening: exact
        assert np.array_equal(bits(wide), bits(ref))
        assert np.array_equal(oracle.f32_to_fp8_bits(wide, fmt), codes)
        # midpoints of neighbouring non-negative codes: exactly representable in fp32, go to the even code
        pos = np.arange(0, top, dtype=np.uint8)
        lo, hi = oracle.fp8_bits_to_f32(pos, fmt).astype(np.float64), oracle.fp8_bits_to_f32(pos + 1, fmt).astype(np.float64)
        mid = ((lo + hi) / 2).astype(np.float32)
        assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)
        got = oracle.f32_to_fp8_bits(mid, fmt)
        assert np.array_equal(got, np.where(pos % 2 == 0, pos, pos + 1))
        assert np.array_equal(oracle.f32_to_fp8_bits(-mid, fmt), np.where(pos % 2 == 0, pos, pos + 1) | 0x80)
        # random and rounding-critical patterns inside the range against torch
        rng = np.random.default_rng(6)
        p = rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)
        x = p.view(np.float32)
        maxv = float(oracle.fp8_bits_to_f32(np.array([top], np.uint8), fmt)[0])
        inside = np.isfinite(x) & (np.abs(x) <= maxv)
        x = np.concatenate([x[inside], (rng.standard_normal(1 << 18) * 2).astype(np.float32),
                            (rng.standard_normal(1 << 18) * 1e-2).astype(np.float32)])
        ref = torch.from_numpy(x.copy()).to(tdt).view(torch.uint8).numpy()
        assert np.array_equal(oracle.f32_to_fp8_bits(x, fmt), ref)
    # the scheme: theta is the widened code, theta_h carries the code, prune first then quantise
    w = np.array([0.3, -1.06, 500.0, 3e-4, 0.0], np.float32)
    out = oracle.cstep_quantize([w], [None], 1.0, ("e4m3",))
    assert out.theta[0].tolist() == [0.3125, -1.0, 448.0, 0.0, 0.0]
    assert out.theta_h[0].tolist() == [0x2A, 0xB8, 0x7E, 0x00, 0x00] and out.mask[0].all()
    out = oracle.cstep_prune([w], [None], 0.6, 1.0, ("e5m2",))
    assert out.theta[0].tolist() == [0.0, -1.0, 512.0, 0.0, 0.0] and out.mask[0].tolist() == [0, 1, 1, 0, 0]


# ---------------------------------------------------------------- criteria and n-D blocks
@pytest.mark.parametrize("crit", ["l2", "l1", "max"])
def test_structure_criteria_closed_forms_and_bruteforce(crit):
    """FilterPrune / NeuronPrune / BlockPrune "based on criteria" (Table 1): the ranked value from
    numpy, the kept set from the O(n^2) rank definition, for slices and for 2-D blocks."""
    rng = np.random.default_rng(12)
    conv = rng.standard_normal((6, 3, 3, 3)).astype(np.float32)
    fc = rng.standard_normal((7, 10)).astype(np.float32)
    lam = [(rng.standard_normal(a.shape) * 0.01).astype(np.float32) for a in (conv, fc)]
    mu = 0.05
    f = {"l2": lambda a: (a * a).sum(1), "l1": lambda a: np.abs(a).sum(1), "max": lambda a: np.abs(a).max(1)}[crit]
    u = [oracle.form_u(a, l, mu).astype(np.float64) for a, l in zip((conv, fc), lam)]
    nu = oracle.structure_values([conv, fc], lam, mu, "structure", criterion=crit)
    ref = np.concatenate([f(u[0].reshape(6, -1)), f(u[1])])
    assert np.allclose(nu, ref, rtol=1e-14, atol=0)
    if crit == "max":
        assert np.array_equal(nu, ref)                         # a maximum has no rounding
    out = oracle.cstep_structured([conv, fc], lam, 0.5, mu, "structure", criterion=crit, fuse=("lambda",))
    keep = brute_keep(nu.view(np.uint64), 13 - 7)
    assert np.array_equal(out.mask[0][:, 0, 0, 0], keep[:6]) and np.array_equal(out.mask[1][:, 0], keep[6:])
    assert np.array_equal(out.mask[0], np.repeat(keep[:6], 27).reshape(conv.shape))
    if crit != "l2":
        assert out.result.tau_norm == pytest.approx(nu[out.result.tau_id], rel=1e-6)
    # 2-D blocks of 3 x 2 on a ragged matrix
    m = rng.standard_normal((8, 7)).astype(np.float32)
    nu = oracle.structure_values([m], [None], 1.0, "block", (3, 2), crit)
    ref = np.array([f(m[3 * r:3 * r + 3, 2 * c:2 * c + 2].astype(np.float64).reshape(1, -1))[0]
                    for r in range(3) for c in range(4)])
    assert np.allclose(nu, ref, rtol=1e-14, atol=0)
    out = oracle.cstep_structured([m], [None], 0.5, 1.0, "block", (3, 2), crit)
    grid = brute_keep(nu.view(np.uint64), 6).reshape(3, 4)
    assert np.array_equal(out.mask[0], np.kron(grid, np.ones((3, 2), np.uint8))[:8, :7])
    # integer data: L1 sums are exact in any order
    ints = rng.integers(-50, 51, size=(5, 40)).astype(np.float32)
    assert oracle.structure_values([ints], [None], 1.0, "neuron", criterion="l1").tolist() == np.abs(ints).sum(1).tolist()
    # with the L2 criterion the specification form is the older call
    a = oracle.cstep_structured([conv, fc], lam, 0.4, mu, "filter", fuse=("lambda",))
    b = oracle.cstep_filter([conv, fc], lam, 0.4, mu, fuse=("lambda",))
    assert all(np.array_equal(x, y) for x, y in zip(a.mask, b.mask)) and a.result.tau_key == b.result.tau_key


@pytest.mark.parametrize("block", [(2, 2, 2), (1, 3, 2), (2, 1, 3, 3), (4, 4), (5,), (3, 2, 1, 2)])
def test_nd_blocks_values_kept_set_and_mask_bruteforce(block):
    """BlockPrune with n-D blocks (Table 1: "n-D blocks of size bs"): every tensor whose rank equals
    the number of block extents is cut into blocks; values from numpy slices in row-major order
    inside the block, kept set by the rank definition, the mask block by block."""
    nd = len(block)
    shape = {1: (23,), 2: (9, 10), 3: (5, 7, 4), 4: (5, 3, 4, 5)}[nd]
    other = {1: (4, 4), 2: (6,), 3: (6, 5), 4: (7, 2, 2)}[nd]
    ws = W.random_set([shape, other, shape], seed=40 + nd, kind="normal", scale=0.3, lam_sigma=1e-2, mu=1e-2)
    s = 0.45
    out = oracle.cstep_structured(ws.w, ws.lam, s, ws.mu, "block", block, "l2", fuse=("lambda",))
    nu = oracle.structure_values(ws.w, ws.lam, ws.mu, "block", block)
    ref, grids = [], []
    for t in (0, 2):
        u = oracle.form_u(ws.w[t], ws.lam[t], ws.mu).astype(np.float64)
        nb = [-(-shape[d] // block[d]) for d in range(nd)]
        grids.append(nb)
        for bidx in itertools.product(*[range(n) for n in nb]):
            sl = tuple(slice(bidx[d] * block[d], (bidx[d] + 1) * block[d]) for d in range(nd))
            acc = 0.0
            for x in u[sl].reshape(-1):                # row-major inside the block
                acc = acc + x * x
            ref.append(acc)
    ref = np.array(ref)
    assert np.array_equal(nu.view(np.uint64), ref.view(np.uint64))
    S = ref.size
    z = int(math.floor(s * S + 0.5))
    keep_s = brute_keep(ref.view(np.uint64), S - z)
    assert out.result.n_units == S and out.result.n_zero == z
    assert out.mask[1].all()                            # another rank: passes through
    sid = 0
    for t, nb in zip((0, 2), grids):
        n = int(np.prod(nb))
        grid = keep_s[sid:sid + n].reshape(nb)
        exp = grid
        for d in range(nd):
            exp = np.repeat(exp, block[d], axis=d)
        exp = exp[tuple(slice(0, shape[d]) for d in range(nd))]
        assert np.array_equal(out.mask[t], exp)
        u = oracle.form_u(ws.w[t], ws.lam[t], ws.mu)
        assert np.array_equal(bits(out.theta[t]), np.where(exp == 1, bits(u), 0))
        sid += n
    assert sid == S
