"""The two load paths of the tensor-core forward (bulk tensor copies for tiles that are contiguous in
the caller's tensors, row-by-row gathers for the rest) and the view-order layout (Q, K, V given and
O, LSE returned in every head's own order, the reordering being left to the producer as Section 3.1
allows), against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def _plan(cfg, rows, cols):
    import paper_2109_04312_b200 as m
    hv = tables.head_view(cfg)
    return m, hv, m.mate_plan(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, hv)


@pytest.mark.parametrize("name,shuffle", [("bert", False), ("bert", True), ("long", False), ("skew", False)])
def test_bulk_copies_and_gathers_give_the_same_bits(name, shuffle):
    # the load path changes how a tile reaches shared memory, not a single arithmetic step
    cfg, rows, cols, info, vals = hp.make_case(name, shuffle=shuffle)
    m, hv, plan = _plan(cfg, rows, cols)
    Q, K, V = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V"))
    O1, L1 = m.mate_attn_fwd(plan, Q, K, V, None, m.IMPL_TCGEN05 | m.FLAG_BULK_TILES)
    O2, L2 = m.mate_attn_fwd(plan, Q, K, V, None, m.IMPL_TCGEN05 | m.FLAG_GATHER_TILES)
    O3, L3 = m.mate_attn_fwd(plan, Q, K, V, None, m.IMPL_TCGEN05)   # the library's own choice
    torch.cuda.synchronize()
    plan.status()
    assert torch.equal(O1, O2) and torch.equal(L1, L2)
    assert torch.equal(O1, O3) and torch.equal(L1, L3)
    with pytest.raises(m.MateError) as e:   # the two loader bits exclude each other
        m.mate_attn_fwd(plan, Q, K, V, None, m.IMPL_TCGEN05 | m.FLAG_BULK_TILES | m.FLAG_GATHER_TILES)
    assert e.value.status == -1
    # and both are the oracle's result (the default path is also covered by the parity tests)
    if name != "long":
        oO, _ = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, 1.0 / np.sqrt(cfg.d))
        hp.assert_close(hp.to_np(O1), oO, *hp.tol(cfg.dtype), "O, bulk copies")
    plan.destroy()


@pytest.mark.parametrize("name,shuffle", [("bert", True), ("medium", False), ("skew", False)])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_view_order_layout(name, shuffle, impl_idx):
    cfg, rows, cols, info, vals = hp.make_case(name, shuffle=shuffle)
    m, hv, plan = _plan(cfg, rows, cols)
    impl = (m.IMPL_SIMT, m.IMPL_TCGEN05)[impl_idx]
    perms = [plan.get(v)[0] for v in (0, 1)]                       # [B, N] per view
    idx = np.stack([perms[int(hv[h])] for h in range(cfg.H)], axis=1)   # [B, H, N]: original position of view position t

    def to_view(x):                                                # x[b, h, idx[b, h, t]] -> position t
        return np.take_along_axis(x, idx.reshape(idx.shape + (1,) * (x.ndim - 3)), axis=2)

    Qv, Kv, Vv = (hp.to_dev(to_view(vals[n]), cfg.dtype) for n in ("Q", "K", "V"))
    scale = 1.0 / np.sqrt(cfg.d)
    O, LSE = m.mate_attn_fwd(plan, Qv, Kv, Vv, scale, impl | m.FLAG_VIEW_ORDER)
    torch.cuda.synchronize()
    plan.status()
    oO, oLSE = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale)
    atol, rtol = hp.tol(cfg.dtype)
    hp.assert_close(hp.to_np(O), to_view(oO), atol, rtol, "O in view order")
    valid = to_view(np.broadcast_to((rows >= 0)[:, None, :], oLSE.shape))
    gL = LSE.cpu().numpy().astype(np.float64)
    hp.assert_close(gL[valid], to_view(oLSE)[valid], atol, rtol, "LSE in view order")
    assert np.all(np.isneginf(gL[~valid])) and np.all(hp.to_np(O)[~valid] == 0)
    # the backward does not take the layout
    with pytest.raises(m.MateError) as e:
        m.mate_attn_bwd(plan, Qv, Kv, Vv, O, LSE, Qv, scale, impl | m.FLAG_VIEW_ORDER)
    assert e.value.status == -2
    plan.destroy()
