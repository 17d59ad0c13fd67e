"""Pins for two further pieces of the CPU oracle (no GPU needed):

* the head-independent "same row OR same column" pattern that the paper describes for its closest
  comparison system (Section 2, related work), selected per head by head_view value 2;
* the per-cell mean of token logits of the cell-selection stage (Section 4.1: S(c) = avg over the
  tokens t of cell c of S(t)).
"""
import math

import numpy as np
import pytest

import oracle
from tests.test_oracle_pins import brute_fwd, rand_qkv, small_table
from workloads import tables


def sat_sets(rows, cols, P):
    """The pattern built token by token as Python sets."""
    N = len(rows)
    valid = [j for j in range(N) if rows[j] >= 0 and cols[j] >= 0]
    sets = []
    for k in range(N):
        if k not in valid:
            sets.append(set())
        elif k < P:
            sets.append(set(valid))
        else:
            sets.append(set(j for j in valid if j < P or rows[j] == rows[k] or cols[j] == cols[k]))
    return sets


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sat_mask_equals_brute_force_sets(seed):
    rows, cols, N = small_table(seed, P=2, n_rows=3, n_cols=4, max_len=2, pad=2)
    M = oracle.mask_sat(rows[0], cols[0], 2)
    sets = sat_sets(rows[0], cols[0], 2)
    for k in range(N):
        assert set(np.nonzero(M[k])[0].tolist()) == sets[k]


def test_sat_mask_is_the_union_of_the_row_and_column_patterns():
    cfg = tables.CONFIGS["bert"]
    rows, cols, info = tables.make_structure(cfg, 5)
    for b in range(2):
        Mr = oracle.mask(rows[b], cols[b], cfg.P, 0)
        Mc = oracle.mask(rows[b], cols[b], cfg.P, 1)
        Ms = oracle.mask_sat(rows[b], cols[b], cfg.P)
        assert np.array_equal(Ms, Mr | Mc)
        assert np.array_equal(Ms, Ms.T)                        # symmetric like the two views
        # pairs: row pairs + column pairs - pairs counted twice (prefix part and the token's own cell)
        both = int((Mr & Mc).sum())
        assert int(Ms.sum()) == int(Mr.sum()) + int(Mc.sum()) - both
    hv = np.asarray([0, 1, 2], np.uint8)
    pairs = oracle.useful_pairs(rows[:1], cols[:1], cfg.P, hv)
    assert pairs[0, 2] == int(oracle.mask_sat(rows[0], cols[0], cfg.P).sum())
    assert pairs[0, 0] == int(oracle.mask(rows[0], cols[0], cfg.P, 0).sum())


def test_sat_head_forward_and_backward_against_loops_and_autograd():
    import torch
    rows, cols, N = small_table(7, P=2, n_rows=3, n_cols=3, max_len=2, pad=1)
    P, d, scale = 2, 4, 0.6
    hv = np.asarray([2, 0, 2], np.uint8)          # mixed with a row head: the per-head switch is pinned too
    Q, K, V, dO = rand_qkv(7, 1, 3, N, d, k=4)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, scale)
    sets = sat_sets(rows[0], cols[0], P)
    for h in (0, 2):
        bO, bL = brute_fwd(Q[0, h], K[0, h], V[0, h], sets, scale)
        np.testing.assert_allclose(O[0, h], bO, rtol=1e-12, atol=1e-14)
        valid = rows[0] >= 0
        np.testing.assert_allclose(LSE[0, h][valid], bL[valid], rtol=1e-12)
    # the row head is untouched by the presence of the other pattern
    O1, _ = oracle.fwd(Q[:, 1:2], K[:, 1:2], V[:, 1:2], rows, cols, P, np.asarray([0], np.uint8), scale)
    assert np.array_equal(O[:, 1:2], O1)
    # backward against autograd through an independent masked softmax over the same sets
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, rows, cols, P, hv, scale)
    M = np.zeros((N, N), dtype=bool)
    for k, A in enumerate(sets):
        M[k, sorted(A)] = True
    q, kk, v = (torch.tensor(x[0, 0], dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    s = (scale * q @ kk.T).masked_fill(~torch.tensor(M), float("-inf"))
    rowvalid = torch.tensor(M.any(-1))[:, None]
    p = torch.where(rowvalid, torch.softmax(torch.where(rowvalid, s, torch.zeros_like(s)), -1), torch.zeros_like(s))
    (p @ v).backward(torch.tensor(dO[0, 0]))
    np.testing.assert_allclose(dQ[0, 0], q.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dK[0, 0], kk.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dV[0, 0], v.grad.numpy(), rtol=1e-10, atol=1e-13)


# ---------------------------------------------------------------- per-cell mean (Section 4.1)

def test_cell_mean_hand_worked():
    # prefix of 2, then cells (row, col): (1,1) x2 tokens, (1,2) x1, (2,1) x3, padding x1
    rows, cols = tables.custom_structure(2, [(1, 1, 2), (1, 2, 1), (2, 1, 3)], 9)
    logits = np.asarray([[9.0, 9.0, 1.0, 2.0, 5.0, -1.0, 0.5, 3.5, 7.0]])
    mean, cnt = oracle.cell_mean(logits, rows, cols, 2, 2, 2)
    assert cnt[0].tolist() == [[0, 0, 0], [0, 2, 1], [0, 3, 0]]
    assert mean[0, 1, 1] == 1.5 and mean[0, 1, 2] == 5.0 and mean[0, 2, 1] == 1.0
    assert mean[0, 0, 0] == 0.0 and mean[0, 2, 2] == 0.0      # no token: count 0, mean 0; prefix excluded


@pytest.mark.parametrize("name", ["tiny", "bert"])
def test_cell_mean_against_per_cell_loops(name):
    cfg = tables.CONFIGS[name]
    rows, cols, info = tables.make_structure(cfg, 3)
    rng = np.random.default_rng(3)
    # shuffle the table tokens of example 0: a cell's tokens need not be adjacent
    sh = cfg.P + rng.permutation(info["n_valid"][0] - cfg.P)
    rows[0, cfg.P:info["n_valid"][0]] = rows[0, sh]
    cols[0, cfg.P:info["n_valid"][0]] = cols[0, sh]
    logits = rng.standard_normal(rows.shape)
    mean, cnt = oracle.cell_mean(logits, rows, cols, cfg.P, cfg.n_rows, cfg.n_cols)
    for b in range(min(cfg.B, 2)):
        cells = {}
        for t in range(cfg.P, rows.shape[1]):
            if rows[b, t] >= 0:
                cells.setdefault((int(rows[b, t]), int(cols[b, t])), []).append(float(logits[b, t]))
        assert int(cnt[b].sum()) == info["n_valid"][b] - cfg.P
        for (r, c), xs in cells.items():
            assert cnt[b, r, c] == len(xs)
            assert math.isclose(mean[b, r, c], math.fsum(xs) / len(xs), rel_tol=1e-12, abs_tol=1e-15)
        assert np.count_nonzero(cnt[b]) == len(cells)
    # a constant logit gives that constant in every non-empty cell
    m1, c1 = oracle.cell_mean(np.full(rows.shape, 2.5), rows, cols, cfg.P, cfg.n_rows, cfg.n_cols)
    assert np.all(m1[c1 > 0] == 2.5) and np.all(m1[c1 == 0] == 0.0)
