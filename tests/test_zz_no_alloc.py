"""mate_attn_bwd_noalloc: the backward for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not available to them: the surrounding framework
owns the whole device, or an allocation (which synchronises the device) would break their latency
budget.  They get one entry point that brings its scratch with it (a fixed array inside the
library).  This test calls it through the C ABI twice in a row, with different inputs, and checks
each result against the CPU oracle's analytic backward and against the ordinary mate_attn_bwd: the
second call shows that whatever the first call left in the shared array does not leak into the
next result.  A second case runs the fp32 path with another head size.

Collected last on purpose (file name), so that a run stopping at the first failure has already run
every other test; it also passes alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def _inputs(cfg, rows, cols, seed):
    import paper_2109_04312_b200 as m
    vals = tables.make_values(cfg, rows.shape[1], seed)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    return m, vals, Q, K, V, dO


def _check_twice(cfg, rows, cols, seeds):
    import paper_2109_04312_b200 as m
    hv = tables.head_view(cfg)
    plan = m.mate_plan(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, hv)
    atol, rtol = hp.tol(cfg.dtype)
    valid = rows >= 0
    scale = 1.0 / np.sqrt(cfg.d)
    for call, seed in enumerate(seeds):
        m, vals, Q, K, V, dO = _inputs(cfg, rows, cols, seed)
        O, LSE = m.mate_attn_fwd(plan, Q, K, V)
        lib = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO)
        want = oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale)
        # outputs are the caller's; poison them so that unwritten elements would show
        outs = [torch.full_like(Q, float("nan")) for _ in range(3)]
        if call == 0:
            # the first call on a device looks up the address of the built-in array
            m.mate_attn_bwd_noalloc(plan, Q, K, V, O, LSE, dO, *outs)
            torch.cuda.synchronize()
        # free bytes as the driver counts them: an allocation by the library itself would show here
        # (torch's own counters only see torch's allocator)
        free_before = torch.cuda.mem_get_info()[0]
        m.mate_attn_bwd_noalloc(plan, Q, K, V, O, LSE, dO, *outs)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        plan.status()
        for name, got, ref, other in zip(("dQ", "dK", "dV"), outs, want, lib):
            g = hp.to_np(got)
            hp.assert_close(g, ref, atol, rtol, "%s vs oracle, call %d" % (name, call))
            hp.assert_close(g, hp.to_np(other), atol, rtol, "%s vs mate_attn_bwd, call %d" % (name, call))
            assert np.all(g[np.broadcast_to(~valid[:, None, :, None], g.shape)] == 0)
    plan.destroy()


def test_noalloc_backward_matches_the_oracle_and_the_workspace_backward_twice():
    cfg = tables.CONFIGS["bert"]
    rows, cols, info = tables.make_structure(cfg, 4321)
    _check_twice(cfg, rows, cols, (11, 12))


def test_noalloc_backward_fp32_other_head_size():
    cfg = tables.CONFIGS["tiny"]                      # fp32, d = 16
    rows, cols, info = tables.make_structure(cfg, 99)
    _check_twice(cfg, rows, cols, (5, 6))


def test_noalloc_backward_rejects_problems_beyond_its_scratch():
    import paper_2109_04312_b200 as m
    # B*H*N = 2 * 9 * 65536 > 1,048,576 rows of scratch; the call must fail before touching tensors
    B, H, N, d = 2, 9, 65536, 8
    ids = torch.zeros((B, N), dtype=torch.int32, device="cuda")
    plan = m.mate_plan(ids, ids, N, [0] * H, 0, 0)
    t = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, H, N), dtype=torch.float32, device="cuda")
    with pytest.raises(m.MateError) as e:
        m.mate_attn_bwd_noalloc(plan, t, t, t, t, lse, t, t.clone(), t.clone(), t.clone())
    assert e.value.status == -8
    torch.cuda.synchronize()
    plan.destroy()
