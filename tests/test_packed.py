"""Packed batches (mate_plan_packed): examples of different length stored one behind the other with no
padding between them.  The examples of a batch are independent (Section 3: the attention sets are
defined inside one example), so the expected values are the oracle's results example by example on that
example's own slice of the packed tensors."""
import numpy as np
import pytest

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def packed_batch(H=4, d=64, dtype="bf16", seed=5, lengths=(517, 64, 1, 900, 0, 333), prefix=(40, 64, 0, 129, 0, 7)):
    """Examples of very different length (one of them empty, one a single token, one only a prefix); the
    last example ends in two padding tokens (negative ids inside an example)."""
    rng = np.random.default_rng(seed)
    rows, cols = [], []
    for L, P in zip(lengths, prefix):
        if L == 0:
            rows.append(np.zeros(0, np.int32))
            cols.append(np.zeros(0, np.int32))
            continue
        nr, nc = int(rng.integers(3, 12)), int(rng.integers(2, 9))
        cells = [(r, c, int(rng.integers(1, 6))) for r in range(1, nr + 1) for c in range(1, nc + 1)]
        while P + sum(c[2] for c in cells) > L:
            cells.pop()
        r_, c_ = tables.custom_structure(P, cells, L)
        # whatever the cells left free becomes table tokens of the last row / first column
        free = r_[0] < 0
        free[:P] = False
        r_[0, free], c_[0, free] = nr, 1
        rows.append(r_[0])
        cols.append(c_[0])
    if lengths[-1] - prefix[-1] >= 4:
        rows[-1][-2:] = -1
        cols[-1][-2:] = -1
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    T = int(cu[-1])
    rng = np.random.default_rng(seed + 1)
    vals = {n: tables.round_to_bf16(rng.standard_normal((H, T, d)).astype(np.float32) * 0.5).astype(np.float64)
            for n in ("Q", "K", "V", "dO")}
    hv = np.array([0, 1] * (H // 2), np.uint8)
    return np.concatenate(rows), np.concatenate(cols), cu, list(prefix), hv, vals


def example(vals, cu, b):
    """[1, H, L, d] views of example b."""
    return {n: np.ascontiguousarray(v[None, :, cu[b]:cu[b + 1]]) for n, v in vals.items()}


def test_packed_plan_is_the_oracles_plan_example_by_example():
    import torch
    import paper_2109_04312_b200 as m
    rows, cols, cu, prefix, hv, _ = packed_batch()
    plan = m.mate_plan_packed(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cu, prefix, hv)
    pairs = plan.useful_pairs()
    assert plan.N == int(np.diff(cu).max())
    for view, ids in ((0, rows), (1, cols)):
        max_id = max(int(ids.max()), 0)
        perm, inv, seg = plan.get(view)
        for b, P in enumerate(prefix):
            L = int(cu[b + 1] - cu[b])
            if L == 0:
                continue
            r, c = rows[None, cu[b]:cu[b + 1]], cols[None, cu[b]:cu[b + 1]]
            operm, oinv, oseg = oracle.plan(r, c, P, view, max_id)
            # inside the example's length the two orders agree; behind it the plan holds padding
            assert np.array_equal(perm[b, :L], operm[0]) and np.array_equal(inv[b, :L], oinv[0])
            assert np.array_equal(perm[b, L:], np.arange(L, plan.N))
            assert np.array_equal(seg[b], oseg[0])
    for b, P in enumerate(prefix):
        if cu[b + 1] == cu[b]:
            assert np.all(pairs[b] == 0)
            continue
        r, c = rows[None, cu[b]:cu[b + 1]], cols[None, cu[b]:cu[b + 1]]
        assert np.array_equal(pairs[b:b + 1], oracle.useful_pairs(r, c, P, hv))
    plan.destroy()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_packed_forward_backward_parity(impl_idx, dtype):
    import torch
    import paper_2109_04312_b200 as m
    if dtype == "f32" and impl_idx == 1:
        pytest.skip("the tensor-core kernels take bf16")
    rows, cols, cu, prefix, hv, vals = packed_batch(dtype=dtype)
    plan = m.mate_plan_packed(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cu, prefix, hv)
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    scale = 0.125
    atol, rtol = hp.tol(dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], dtype) for n in ("Q", "K", "V", "dO"))
    sentinel = 7.0
    O = torch.full_like(Q, sentinel)
    LSE = torch.full(Q.shape[:2], sentinel, dtype=torch.float32, device=Q.device)
    m.mate_attn_fwd(plan, Q, K, V, scale, impl, out=O, lse=LSE)
    dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    gO, gL = hp.to_np(O), LSE.cpu().numpy().astype(np.float64)
    assert not np.any(gL == sentinel) and not np.any(gO == sentinel)   # every row of every example was written
    grads = [hp.to_np(g) for g in (dQ, dK, dV)]
    for b, P in enumerate(prefix):
        if cu[b + 1] == cu[b]:
            continue
        sl = slice(cu[b], cu[b + 1])
        r, c = rows[None, sl], cols[None, sl]
        ex = example(vals, cu, b)
        oO, oL = oracle.fwd(ex["Q"], ex["K"], ex["V"], r, c, P, hv, scale)
        og = oracle.bwd(ex["Q"], ex["K"], ex["V"], ex["dO"], r, c, P, hv, scale)
        valid = np.broadcast_to((r >= 0)[:, None, :], oL.shape)
        hp.assert_close(gO[None, :, sl], oO, atol, rtol, "O of example %d" % b)
        hp.assert_close(gL[None, :, sl][valid], oL[valid], atol, rtol, "LSE of example %d" % b)
        for nm, g, o in zip(("dQ", "dK", "dV"), grads, og):
            hp.assert_close(g[None, :, sl], o, atol, rtol, "%s of example %d" % (nm, b))
    plan.destroy()


def test_packed_equals_padded():
    """The same examples once packed and once padded to the longest: bit-identical results on the rows that
    exist in both (the kernels run the same plan; only the addressing differs)."""
    import torch
    import paper_2109_04312_b200 as m
    rows, cols, cu, prefix, hv, vals = packed_batch(lengths=(400, 257, 130), prefix=(20, 0, 130))
    B, H, d = len(prefix), len(hv), 64
    N = int(np.diff(cu).max())
    prow = np.full((B, N), -1, np.int32)
    pcol = np.full((B, N), -1, np.int32)
    pad = {n: np.zeros((B, H, N, d)) for n in vals}
    for b in range(B):
        L = cu[b + 1] - cu[b]
        prow[b, :L], pcol[b, :L] = rows[cu[b]:cu[b + 1]], cols[cu[b]:cu[b + 1]]
        for n in vals:
            pad[n][b, :, :L] = vals[n][:, cu[b]:cu[b + 1]]
    packed = m.mate_plan_packed(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cu, prefix, hv)
    padded = m.mate_plan_varlen(torch.from_numpy(prow).cuda(), torch.from_numpy(pcol).cuda(), prefix, hv)
    for impl in (m.IMPL_SIMT, m.IMPL_TCGEN05):
        a = [hp.to_dev(vals[n], "bf16") for n in ("Q", "K", "V", "dO")]
        p = [hp.to_dev(pad[n], "bf16") for n in ("Q", "K", "V", "dO")]
        Oa, La = m.mate_attn_fwd(packed, *a[:3], 0.125, impl)
        Op, Lp = m.mate_attn_fwd(padded, *p[:3], 0.125, impl)
        ga = m.mate_attn_bwd(packed, *a[:3], Oa, La, a[3], 0.125, impl)
        gp = m.mate_attn_bwd(padded, *p[:3], Op, Lp, p[3], 0.125, impl)
        torch.cuda.synchronize()
        for b in range(B):
            L = cu[b + 1] - cu[b]
            assert torch.equal(Oa[:, cu[b]:cu[b + 1]], Op[b, :, :L])
            assert torch.equal(La[:, cu[b]:cu[b + 1]], Lp[b, :, :L])
            for x, y in zip(ga, gp):   # no gradient is accumulated across CTAs: the same bits here too
                assert torch.equal(x[:, cu[b]:cu[b + 1]], y[b, :, :L])
    packed.status()
    padded.status()
    packed.destroy()
    padded.destroy()


def test_packed_rejects_bad_arguments():
    import torch
    import paper_2109_04312_b200 as m
    rows = torch.tensor([0, 0, 1, 1, 0, 1, 1, 2], dtype=torch.int32).cuda()
    cols = torch.tensor([0, 0, 1, 2, 0, 1, 2, 1], dtype=torch.int32).cuda()
    lib = m.api._load()
    import ctypes as C

    def status(cu, prefix):
        cu, pf = np.asarray(cu, np.int32), np.asarray(prefix, np.int32)
        hv = np.array([0, 1], np.uint8)
        h = C.c_void_p()
        rc = lib.mate_plan_packed(rows.data_ptr(), cols.data_ptr(), len(pf), cu.ctypes.data, pf.ctypes.data,
                                  hv.ctypes.data, 2, 2, 2, None, C.byref(h))
        if rc == 0:
            lib.mate_plan_destroy(h)
        return rc

    assert status([0, 4, 8], [2, 1]) == 0
    assert status([1, 4, 8], [2, 1]) == -1   # does not start at 0
    assert status([0, 5, 4], [2, 1]) == -1   # decreasing
    assert status([0, 4, 8], [5, 1]) == -1   # prefix longer than the example
    assert status([0, 4, 8], [3, 1]) == -1   # a non-zero id inside the first example's prefix
    plan = m.mate_plan_packed(rows, cols, [0, 4, 8], [2, 1], [0, 1])
    q = torch.zeros(2, 8, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.MateError) as e:
        m.mate_attn_fwd(plan, q, q, q, 0.125, m.IMPL_AUTO | m.FLAG_VIEW_ORDER)
    assert e.value.status == -2
    plan.destroy()
