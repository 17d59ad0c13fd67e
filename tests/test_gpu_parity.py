"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def mate():
    import paper_2109_04312_b200 as m
    return m


def impls_for(cfg):
    m = mate()
    if cfg.dtype == "bf16" and cfg.d == 64:
        return [m.IMPL_SIMT, m.IMPL_TCGEN05]
    return [m.IMPL_SIMT]


def make_plan(cfg, rows, cols, head_view=None):
    m = mate()
    hv = tables.head_view(cfg) if head_view is None else head_view
    r = torch.from_numpy(rows).cuda()
    c = torch.from_numpy(cols).cuda()
    return m.mate_plan(r, c, cfg.P, hv, max(int(rows.max()), 0), max(int(cols.max()), 0)), hv


# -------------------------------------------------------------------------------- plan (bit exact)

@pytest.mark.parametrize("name", ["tiny", "bert", "medium", "long", "skew"])
@pytest.mark.parametrize("shuffle", [False, True])
def test_plan_bit_exact(name, shuffle):
    cfg, rows, cols, info, _ = hp.make_case(name, shuffle=shuffle)
    plan, hv = make_plan(cfg, rows, cols)
    for view, ids in ((0, rows), (1, cols)):
        max_id = max(int(ids.max()), 0)
        perm, inv, seg = plan.get(view)
        operm, oinv, oseg = oracle.plan(rows, cols, cfg.P, view, max_id)
        assert np.array_equal(perm, operm)
        assert np.array_equal(inv, oinv)
        assert np.array_equal(seg, oseg)
    assert np.array_equal(plan.useful_pairs(), oracle.useful_pairs(rows, cols, cfg.P, hv))
    plan.destroy()


def test_plan_edge_cases():
    m = mate()
    cases = []
    # no prefix, ragged length, id 0 used by table tokens, interleaved padding, large sparse ids
    rows = np.asarray([[0, 0, 3, 3, -1, 7, 0, 7, 3, -1, 900, 1, 1]], np.int32)
    cols = np.asarray([[5, 4, 5, 0, -1, 0, 4, 5, 5, -1, 2, 2, 0]], np.int32)
    cases.append((rows, cols, 0))
    # only a prefix
    cases.append((np.zeros((2, 37), np.int32), np.zeros((2, 37), np.int32), 37))
    # prefix followed by padding only
    r = np.full((1, 70), -1, np.int32)
    r[0, :5] = 0
    cases.append((r, r.copy(), 5))
    # everything padding, P = 0
    cases.append((np.full((1, 33), -1, np.int32), np.full((1, 33), -1, np.int32), 0))
    # many distinct ids (histogram wider than the shared-memory path)
    rng = np.random.default_rng(0)
    r = rng.integers(0, 6000, size=(2, 3000)).astype(np.int32)
    c = rng.integers(0, 50, size=(2, 3000)).astype(np.int32)
    r[:, :10] = 0
    c[:, :10] = 0
    cases.append((r, c, 10))
    for rows, cols, P in cases:
        mr, mc = max(int(rows.max()), 0), max(int(cols.max()), 0)
        plan = m.mate_plan(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), P, [0, 1, 1], mr, mc)
        for view, max_id in ((0, mr), (1, mc)):
            perm, inv, seg = plan.get(view)
            operm, oinv, oseg = oracle.plan(rows, cols, P, view, max_id)
            assert np.array_equal(perm, operm) and np.array_equal(inv, oinv) and np.array_equal(seg, oseg)
        assert np.array_equal(plan.useful_pairs(), oracle.useful_pairs(rows, cols, P, np.asarray([0, 1, 1], np.uint8)))
        plan.destroy()


def test_plan_rejects_bad_ids():
    m = mate()

    def status_of(rows, cols, P, mr=5, mc=5):
        try:
            m.mate_plan(torch.tensor(rows, dtype=torch.int32).cuda(), torch.tensor(cols, dtype=torch.int32).cuda(),
                        P, [0, 1], mr, mc)
        except m.MateError as e:
            return e.status
        return 0

    assert status_of([[0, 0, 1, 1]], [[0, 0, 1, 2]], 2) == 0
    assert status_of([[0, 1, 1, 1]], [[0, 0, 1, 2]], 2) == -1      # non-zero id inside the prefix
    assert status_of([[0, 0, -1, 1]], [[0, 0, 1, 2]], 2) == -1     # padding flags disagree
    assert status_of([[0, 0, 9, 1]], [[0, 0, 1, 2]], 2) == -1      # id above max_row_id
    assert status_of([[0, -1, 1, 1]], [[0, -1, 1, 2]], 2) == -1    # padding inside the prefix
    assert status_of([[0, 0, 1, 1]], [[0, 0, 1, 2]], 5) == -1      # prefix longer than the sequence


# -------------------------------------------------------------------------------- forward / backward

def run_case(cfg, rows, cols, vals, impl, head_view=None, backward=None, scale=None, unit_grads=False):
    """Forward (and backward) through the C ABI against the oracle.  unit_grads: for inputs much
    larger than the usual N(0,1)/2 -- whose gradients would be tens of times larger too, while the
    tolerance has a fixed absolute part -- dO is multiplied by a power of two chosen so that dQ keeps
    its usual size (root mean square about 1/4).  The backward is linear in dO and a power of two is
    exact, so the oracle's gradients are scaled by the same factor."""
    m = mate()
    plan, hv = make_plan(cfg, rows, cols, head_view)
    scale = (1.0 / np.sqrt(cfg.d)) if scale is None else scale
    atol, rtol = hp.tol(cfg.dtype)
    Q, K, V, dO = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V", "dO"))
    O, LSE = m.mate_attn_fwd(plan, Q, K, V, scale, impl)
    torch.cuda.synchronize()
    plan.status()
    oO, oLSE = oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale)
    valid = rows >= 0                                    # [B, N]
    vmask = np.broadcast_to(valid[:, None, :], oLSE.shape)
    gO, gLSE = hp.to_np(O), LSE.detach().cpu().numpy().astype(np.float64)
    hp.assert_close(gO, oO, atol, rtol, "O")
    assert np.all(gO[~vmask] == 0), "padding rows of O must be exact zeros"
    assert np.all(np.isneginf(gLSE[~vmask])), "padding rows of LSE must be -inf"
    hp.assert_close(gLSE[vmask], oLSE[vmask], atol, rtol, "LSE")
    do_bwd = cfg.backward if backward is None else backward
    if do_bwd:
        odQ, odK, odV = oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale)
        if unit_grads:
            rms = float(np.sqrt(np.mean(np.square(odQ[np.broadcast_to(valid[:, None, :, None], odQ.shape)]))))
            f = 2.0 ** min(0, int(np.floor(np.log2(0.25 / max(rms, 1e-30)))))
            dO = (dO.float() * f).to(dO.dtype)
            odQ, odK, odV = odQ * f, odK * f, odV * f
        dQ, dK, dV = m.mate_attn_bwd(plan, Q, K, V, O, LSE, dO, scale, impl)
        torch.cuda.synchronize()
        plan.status()
        for nm, g, o in (("dQ", dQ, odQ), ("dK", dK, odK), ("dV", dV, odV)):
            g = hp.to_np(g)
            hp.assert_close(g, o, atol, rtol, nm)
            assert np.all(g[np.broadcast_to(~valid[:, None, :, None], g.shape)] == 0), nm + " padding rows"
    plan.destroy()
    return gO, gLSE


@pytest.mark.parametrize("seed", [1234, 1, 2])
def test_tiny_fp32(seed):
    cfg, rows, cols, info, vals = hp.make_case("tiny", seed_structure=seed, seed_values=seed + 1)
    run_case(cfg, rows, cols, vals, mate().IMPL_SIMT, backward=True)


@pytest.mark.parametrize("name", ["bert", "medium", "long", "skew"])
@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
@pytest.mark.parametrize("seed", [1234, 21, 22])
def test_config_parity(name, impl_idx, seed):
    # three table structures (and value draws) per configuration; seed 1234 is the benchmark's
    cfg, rows, cols, info, vals = hp.make_case(name, seed_structure=seed, seed_values=seed + 4444)
    run_case(cfg, rows, cols, vals, impls_for(cfg)[impl_idx])


@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
@pytest.mark.parametrize("seed", [7, 8])
def test_shuffled_tokens(impl_idx, seed):
    # table tokens in random order: both views need a real gather / scatter
    cfg, rows, cols, info, vals = hp.make_case("bert", seed_structure=seed, seed_values=seed, shuffle=True)
    run_case(cfg, rows, cols, vals, impls_for(cfg)[impl_idx])


def custom_case(P, cells, N, B=1, H=2, d=64, dtype="bf16", seed=0, scale_values=0.5):
    rows, cols = tables.custom_structure(P, cells, N)
    rows = np.repeat(rows, B, axis=0)
    cols = np.repeat(cols, B, axis=0)
    cfg = tables.TableConfig("custom", B, H, H // 2, d, N, P, 0, 0, "uniform", 1, 1, dtype, scale_values)
    vals = tables.make_values(cfg, N, seed)
    return cfg, rows, cols, vals


@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_edge_structures(impl_idx):
    cases = []
    # no prefix: table tokens see only their own segment; ragged N; segments of length 1
    cases.append(custom_case(0, [(r, c, 1 + (r * c) % 3) for r in range(1, 9) for c in range(1, 5)], 77))
    # prefix only (no table token), with padding behind it
    cases.append(custom_case(150, [], 200))
    # prefix not a multiple of the tile, one long segment crossing several tiles, tail padding
    cases.append(custom_case(70, [(1, 1, 300), (2, 1, 5), (2, 2, 260)], 700))
    # one row spanning the table: row heads are dense attention
    cases.append(custom_case(9, [(1, c, 17) for c in range(1, 12)], 9 + 17 * 11))
    # header row numbered 0 (table tokens with id 0)
    cases.append(custom_case(5, [(0, 1, 3), (0, 2, 4), (1, 1, 2), (1, 2, 6)], 40))
    for cfg, rows, cols, vals in cases:
        run_case(cfg, rows, cols, vals, impls_for(cfg)[impl_idx], backward=True)


@pytest.mark.parametrize("impl_idx", [0, 1], ids=["simt", "tc"])
def test_single_view_head_sets(impl_idx):
    # ablations of the paper drop all row heads or all column heads: one view has no head
    cfg, rows, cols, vals = custom_case(20, [(r, c, 2) for r in range(1, 30) for c in range(1, 6)], 330, H=3)
    for hv in ([0, 0, 0], [1, 1, 1], [1, 0, 1]):
        run_case(cfg, rows, cols, vals, impls_for(cfg)[impl_idx], head_view=np.asarray(hv, np.uint8), backward=True)


def test_other_head_dims_simt():
    for d, dtype in ((8, "f32"), (32, "bf16"), (128, "bf16"), (40, "f32")):
        cfg, rows, cols, vals = custom_case(6, [(r, c, 2) for r in range(1, 5) for c in range(1, 4)], 35, d=d, dtype=dtype)
        run_case(cfg, rows, cols, vals, mate().IMPL_SIMT, backward=True)


def test_forward_is_reproducible_and_stays_in_bounds():
    m = mate()
    cfg, rows, cols, info, vals = hp.make_case("medium")
    plan, hv = make_plan(cfg, rows, cols)
    Q, K, V = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V"))
    n = Q.numel()
    for impl in impls_for(cfg):
        # canaries on both sides of the outputs
        buf = torch.full((n + 4096,), 7.0, dtype=torch.bfloat16, device="cuda")
        lbuf = torch.full((cfg.B * cfg.H * info["N"] + 2048,), 7.0, dtype=torch.float32, device="cuda")
        O = buf[2048:2048 + n].view_as(Q)
        L = lbuf[1024:1024 + cfg.B * cfg.H * info["N"]].view(cfg.B, cfg.H, info["N"])
        m.mate_attn_fwd(plan, Q, K, V, None, impl, out=O, lse=L)
        O1, L1 = O.clone(), L.clone()
        m.mate_attn_fwd(plan, Q, K, V, None, impl, out=O, lse=L)
        torch.cuda.synchronize()
        assert torch.equal(O1, O) and torch.equal(L1, L)
        assert torch.all(buf[:2048] == 7.0) and torch.all(buf[2048 + n:] == 7.0)
        assert torch.all(lbuf[:1024] == 7.0) and torch.all(lbuf[1024 + L.numel():] == 7.0)
    plan.destroy()


def test_argument_errors_launch_nothing():
    m = mate()
    cfg, rows, cols, vals = custom_case(4, [(1, 1, 4), (2, 1, 4)], 16, d=64)
    plan, hv = make_plan(cfg, rows, cols)
    Q, K, V = (hp.to_dev(vals[n], "bf16") for n in ("Q", "K", "V"))

    def status(fn):
        try:
            fn()
        except m.MateError as e:
            return e.status
        return 0

    # misaligned pointer
    flat = torch.zeros(Q.numel() + 8, dtype=torch.bfloat16, device="cuda")
    Qm = flat[1:1 + Q.numel()].view_as(Q)
    assert status(lambda: m.mate_attn_fwd(plan, Qm, K, V)) == -3
    # unsupported head dim for the tensor-core path
    Q32 = torch.zeros(1, 2, 16, 32, dtype=torch.bfloat16, device="cuda")
    assert status(lambda: m.mate_attn_fwd(plan, Q32, Q32, Q32, impl=m.IMPL_TCGEN05)) == -2
    # head dim not a multiple of 8
    Q12 = torch.zeros(1, 2, 16, 12, dtype=torch.float32, device="cuda")
    assert status(lambda: m.mate_attn_fwd(plan, Q12, Q12, Q12)) == -2
    # backward without enough workspace
    O, LSE = m.mate_attn_fwd(plan, Q, K, V)
    tiny_ws = torch.zeros(256, dtype=torch.uint8, device="cuda")[:8]
    assert status(lambda: m.mate_attn_bwd(plan, Q, K, V, O, LSE, Q, workspace=tiny_ws)) == -7
    torch.cuda.synchronize()
    plan.destroy()


def test_expired_wait_is_reported_once_and_the_plan_stays_usable():
    # No kernel of the library is made to wait in vain: a one-thread test kernel runs the same bounded
    # wait with a limit of a few tries on a barrier nothing arrives on, gives up and raises the plan's
    # time-out word the way the attention kernels would.
    m = mate()
    cfg, rows, cols, info, vals = hp.make_case("bert")
    plan, hv = make_plan(cfg, rows, cols)
    Q, K, V = (hp.to_dev(vals[n], cfg.dtype) for n in ("Q", "K", "V"))
    O0, L0 = m.mate_attn_fwd(plan, Q, K, V)
    torch.cuda.synchronize()
    plan.status()                                   # nothing has expired so far
    plan.debug_expire_wait()
    with pytest.raises(m.MateError) as e:
        plan.status()
    assert e.value.status == -5                     # MATE_ERR_TIMEOUT
    plan.status()                                   # reported once, then clear again
    O1, L1 = m.mate_attn_fwd(plan, Q, K, V)         # the plan is still good
    torch.cuda.synchronize()
    plan.status()
    assert torch.equal(O0, O1) and torch.equal(L0, L1)
    plan.destroy()
