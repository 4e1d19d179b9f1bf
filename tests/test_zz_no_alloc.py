"""The allocation-free pruning entry point against the regular one.

``condensa_cstep_prune_noalloc`` exists for programs that cannot let a library
allocate device memory: a pool allocator owns the whole device, or a
latency-critical loop cannot take the device-wide synchronisation that
cudaMalloc / cudaFree bring. It keeps its scratch in a fixed array inside the
library, shared by all calls, so the test runs it twice in a row on different
inputs: the second call sees the first one's leftovers in that array and must
still match ``condensa_cstep_prune`` bit for bit.

This file sorts last on purpose, so that a run stopping at the first failure
has already gone through every other test.
"""
import numpy as np
import pytest

from paper_1911_02497_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _bits(a):
    return np.ascontiguousarray(a).view(np.uint8)


def _both(ctx, ws, sparsity, fuse, elem_offset=0):
    """Outputs of the regular and of the allocation-free call on the same input."""
    from paper_1911_02497_b200 import cstep
    from paper_1911_02497_b200.device_set import DeviceSet
    ref = DeviceSet(ws.w, ws.lam, elem_offset=elem_offset)
    ref.poison_outputs()
    ref.run(ctx, "prune", sparsity, ws.mu, fuse)
    want = ref.fetch()
    ds = DeviceSet(ws.w, ws.lam, elem_offset=elem_offset)
    ds.poison_outputs()
    cstep.cstep_prune_noalloc(ds.table, sparsity, ws.mu, fuse)
    got = ds.fetch()
    return got, want


def test_noalloc_prune_matches_regular_entry_point_twice_in_a_row():
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    try:
        # first call: close to the size limit, threshold found through list passes
        a = W.random_set([(1000003,)], seed=11, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
        # second call: smaller, other sparsity, unaligned buffers, many ties - it starts from
        # the scratch contents the first call left behind
        b = W.random_set([(70001,)], seed=12, kind="normal", scale=4.0, lam_sigma=0.0, mu=1.0)
        b.w[0] = np.round(b.w[0])
        cases = [(a, 0.9, ("fp16", "lambda", "penalty"), 0), (b, 0.37, ("lambda",), 3),
                 (a, 0.999, ("lambda",), 0)]
        for ws, s, fuse, off in cases:
            got, want = _both(ctx, ws, s, fuse, off)
            for key in ("theta", "mask", "lam", "theta_h") + (("grad",) if "penalty" in fuse else ()):
                assert np.array_equal(_bits(got[key][0]), _bits(want[key][0])), (key, s)
            assert int((got["mask"][0] == 0).sum()) == int(np.floor(s * ws.numel + 0.5))
    finally:
        ctx.close()


def test_noalloc_at_the_size_limit_allocates_nothing_and_reports_status():
    """The largest accepted input (it takes the largest scratch layout), the device's free
    memory across a steady-state call (the library must not have allocated), and the status
    call that tells whether the device-side checks of the last call passed."""
    import torch
    from paper_1911_02497_b200 import cstep
    ctx = cstep.Context(0)
    try:
        ws = W.random_set([(cstep.NOALLOC_MAX_NUMEL,)], seed=13, kind="normal", scale=0.05, lam_sigma=1e-2, mu=1e-2)
        got, want = _both(ctx, ws, 0.95, ("lambda", "penalty"))
        cstep.noalloc_status()
        for key in ("theta", "mask", "lam", "grad"):
            assert np.array_equal(_bits(got[key][0]), _bits(want[key][0])), key
        from paper_1911_02497_b200.device_set import DeviceSet
        ds = DeviceSet(ws.w, ws.lam)
        cstep.cstep_prune_noalloc(ds.table, 0.5, ws.mu, ("lambda",))      # any first-use set-up is behind us now
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info(0)
        ds.reset_lambda()
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info(0)
        cstep.cstep_prune_noalloc(ds.table, 0.5, ws.mu, ("lambda",))
        cstep.noalloc_status()
        free2, _ = torch.cuda.mem_get_info(0)
        assert free2 == free1, (free0, free1, free2)
    finally:
        ctx.close()


def test_noalloc_rejects_what_does_not_fit():
    import torch
    from paper_1911_02497_b200 import cstep
    n = cstep.NOALLOC_MAX_NUMEL + 1
    w = torch.zeros(n, device="cuda:0")
    th = torch.full((n,), 5.0, device="cuda:0")
    tab = cstep.tensor_table([w], None, [th], shapes=[(n,)])
    with pytest.raises(cstep.CondensaError) as e:
        cstep.cstep_prune_noalloc(tab, 0.5, 1e-3)
    assert e.value.code == cstep.ERR_TOO_LARGE and "NOALLOC_MAX_NUMEL" in str(e.value)
    torch.cuda.synchronize()
    assert bool((th == 5.0).all())                      # nothing was written
    tab = cstep.tensor_table([w[:16]], None, [th[:16]], shapes=[(16,)])
    with pytest.raises(cstep.CondensaError) as e:
        cstep.cstep_prune_noalloc(tab, 1.5, 1e-3)
    assert e.value.code == cstep.ERR_INVALID_ARG
