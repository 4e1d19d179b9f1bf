"""Host logic that needs no GPU: the workspace query plans a call (work decomposition, candidate
list, journal, tile configuration) without touching a device, so its answers can be checked
here for the properties the planning has to have."""
import ctypes as C

import pytest


def _table(shapes, base=1 << 30, with_lam=True):
    """A tensor table over made-up, 256-byte aligned device addresses (never dereferenced)."""
    from paper_1911_02497_b200 import cstep
    addr, w, lam, theta, mask = base, [], [], [], []
    for shp in shapes:
        n = 1
        for d in shp:
            n *= d
        step = (4 * n + 255) // 256 * 256 + 256
        w.append(addr); lam.append(addr + step); theta.append(addr + 2 * step); mask.append(addr + 3 * step)
        addr += 4 * step
    return cstep.tensor_table(w, lam if with_lam else None, theta, mask, shapes=shapes), len(shapes)


def _block_spec(bh, bw):
    from paper_1911_02497_b200 import cstep
    return cstep.StructureSpec(cstep.SPEC_BLOCKS, 0, cstep.CRITERIA["l2"], 2, (bh, bw, 1, 1))


def test_workspace_grows_with_the_list_and_is_a_multiple_of_a_mebibyte():
    from paper_1911_02497_b200 import cstep
    sizes = []
    for rows in (1000, 4000, 16000):
        tab, T = _table([(rows, 1500), (1500,)])
        sizes.append(cstep.workspace_bytes(cstep.OP_PRUNE, tab, T, ("lambda",)))
    assert sizes[0] < sizes[1] < sizes[2]
    assert all(s % (1 << 20) == 0 for s in sizes)


def test_sampling_switch_changes_what_a_call_reserves():
    """The single-pass route keeps a journal of original multipliers beside the candidate list;
    CONDENSA_NO_SAMPLING does without it."""
    from paper_1911_02497_b200 import cstep
    tab, T = _table([(8000, 1500), (6000, 1500)])
    with_s = cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, ("lambda",))
    without = cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, ("lambda", "no_sampling"))
    assert with_s > without > 0


def test_five_by_five_blocks_reserve_for_both_routes():
    """5 x 5 blocks may take their single-pass kernel (journal of 25 floats per listed block) or
    the route over the norm array (8 bytes per block): the query covers the larger of the two;
    a shape the kernel is not built for needs the norm array only."""
    from paper_1911_02497_b200 import cstep
    tab, T = _table([(8000, 1500), (6000, 1500)])
    s55, s73 = _block_spec(5, 5), _block_spec(7, 3)
    b55 = cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, ("lambda",), C.byref(s55))
    b55_ns = cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, ("lambda", "no_sampling"), C.byref(s55))
    b73 = cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, ("lambda",), C.byref(s73))
    assert b55 > b55_ns > 0 and b73 > 0
    # unaligned matrices (width no multiple of 4) cannot take the tiled kernel: no journal is reserved
    tab_u, T_u = _table([(8000, 1501), (6000, 1501)])
    assert cstep.workspace_bytes(cstep.OP_BLOCK, tab_u, T_u, ("lambda",), C.byref(s55)) == \
        cstep.workspace_bytes(cstep.OP_BLOCK, tab_u, T_u, ("lambda", "no_sampling"), C.byref(s55))


def test_bad_queries_are_refused():
    from paper_1911_02497_b200 import cstep
    tab, T = _table([(64, 64)])
    with pytest.raises(cstep.CondensaError):
        cstep.workspace_bytes(99, tab, T)
    bad = cstep.StructureSpec(cstep.SPEC_BLOCKS, 0, cstep.CRITERIA["l2"], 7, (5, 5, 1, 1))
    with pytest.raises(cstep.CondensaError):
        cstep.workspace_bytes(cstep.OP_BLOCK, tab, T, (), C.byref(bad))
