"""Pins for the CPU oracle: closed forms, brute force, invariants, library routines and finite
differences.  Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign
or index, transposed operand, wrong set) fails at least one of them.  No GPU needed."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from workloads import tables

HERE = os.path.dirname(os.path.abspath(__file__))


def small_table(seed, P=3, n_rows=3, n_cols=3, max_len=3, pad=2, B=1):
    rng = np.random.default_rng(seed)
    rr, cc = [], []
    for _ in range(B):
        cells = [(r, c, int(rng.integers(1, max_len + 1)))
                 for r in range(1, n_rows + 1) for c in range(1, n_cols + 1)]
        rr.append(cells)
    n = max(P + sum(l for _, _, l in cells) for cells in rr) + pad
    rows = np.concatenate([tables.custom_structure(P, cells, n)[0] for cells in rr])
    cols = np.concatenate([tables.custom_structure(P, cells, n)[1] for cells in rr])
    return rows, cols, n


def rand_qkv(seed, B, H, N, d, k=3):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((B, H, N, d)) for _ in range(k)]


def brute_sets(row_ids, col_ids, P, view):
    """A_k of Section 3 built token by token as Python sets (padding removed)."""
    ids = row_ids if view == 0 else col_ids
    N = len(ids)
    valid = [j for j in range(N) if ids[j] >= 0]
    Qset = set(j for j in range(P) if ids[j] >= 0)
    sets = []
    for k in range(N):
        if ids[k] < 0:
            sets.append(set())
        elif k < P:
            sets.append(set(valid))
        else:
            sets.append(Qset | set(j for j in valid if j >= P and ids[j] == ids[k]))
    return sets


def brute_fwd(Q, K, V, sets, scale):
    """Per-token loops in Python floats over explicit sets (one head)."""
    N, d = Q.shape
    O = np.zeros((N, d))
    LSE = np.full(N, -np.inf)
    for k in range(N):
        A = sorted(sets[k])
        if not A:
            continue
        s = [scale * sum(Q[k, e] * K[j, e] for e in range(d)) for j in A]
        m = max(s)
        w = [math.exp(x - m) for x in s]
        Z = sum(w)
        for wj, j in zip(w, A):
            for e in range(d):
                O[k, e] += wj / Z * V[j, e]
        LSE[k] = m + math.log(Z)
    return O, LSE


# ---------------------------------------------------------------- mask / pattern

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_mask_equals_brute_force_sets(seed):
    rows, cols, N = small_table(seed)
    for view in (0, 1):
        M = oracle.mask(rows[0], cols[0], 3, view)
        sets = brute_sets(rows[0], cols[0], 3, view)
        for k in range(N):
            assert set(np.nonzero(M[k])[0].tolist()) == sets[k]


def test_mask_invariants_and_popcount():
    cfg = tables.CONFIGS["bert"]
    rows, cols, info = tables.make_structure(cfg, seed=7)
    hv = tables.head_view(cfg)
    pairs = oracle.useful_pairs(rows, cols, cfg.P, hv)
    for b in range(cfg.B):
        nv = info["n_valid"][b]
        for view, ids in ((0, rows[b]), (1, cols[b])):
            M = oracle.mask(rows[b], cols[b], cfg.P, view)
            valid = ids >= 0
            # every valid token attends to itself; the first token attends to and from everything
            assert np.all(np.diag(M)[valid] == 1) and np.all(np.diag(M)[~valid] == 0)
            assert np.all(M[0, valid] == 1) and np.all(M[valid, 0] == 1)
            assert np.all(M[~valid, :] == 0) and np.all(M[:, ~valid] == 0)
            assert np.array_equal(M, M.T)
            # O(ng + nb) count: P * n_valid + sum_s L_s (L_s + P)
            L = np.bincount(ids[cfg.P:nv])
            expect = cfg.P * nv + int(np.sum(L * (L + cfg.P)))
            assert int(M.sum()) == expect
            for h in np.nonzero(hv == view)[0]:
                assert pairs[b, h] == expect


def test_table_token_with_id_zero_is_a_table_token():
    # header row numbered 0: a segment of its own, not part of the prefix
    rows, cols = tables.custom_structure(2, [(0, 1, 2), (0, 2, 1), (1, 1, 2), (1, 2, 1)])
    M = oracle.mask(rows[0], cols[0], 2, 0)
    # token 2 (row 0) sees prefix {0,1} and row-0 tokens {2,3,4}; not row-1 tokens {5,6,7}
    assert M[2].tolist() == [1, 1, 1, 1, 1, 0, 0, 0]
    assert M[5].tolist() == [1, 1, 0, 0, 0, 1, 1, 1]


# ---------------------------------------------------------------- forward values

def test_hand_worked_example():
    with open(os.path.join(HERE, "golden", "hand_worked_attention.json")) as f:
        g = json.load(f)
    a = np.asarray(g["a"], dtype=np.float64)
    N = len(a)
    Q = np.ones((1, 2, N, 1))
    K = np.broadcast_to(np.log(a)[None, None, :, None], (1, 2, N, 1)).copy()
    V = np.broadcast_to(np.asarray(g["v"], np.float64)[None, None, :, None], (1, 2, N, 1)).copy()
    rows = np.asarray([g["row_ids"]], np.int32)
    cols = np.asarray([g["col_ids"]], np.int32)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, g["P"], np.asarray([0, 1], np.uint8), 1.0)
    for h, key in ((0, "row_head"), (1, "col_head")):
        expO = np.asarray(g[key]["O_num"], np.float64) / np.asarray(g[key]["O_den"], np.float64)
        np.testing.assert_allclose(O[0, h, :, 0], expO, rtol=1e-13)
        np.testing.assert_allclose(LSE[0, h], np.log(np.asarray(g[key]["Z"], np.float64)), rtol=1e-13)


@pytest.mark.parametrize("seed", [0, 1])
def test_fwd_equals_brute_force_loops(seed):
    rows, cols, N = small_table(seed, B=2)
    H, d, P = 2, 4, 3
    Q, K, V = rand_qkv(seed, 2, H, N, d)
    hv = np.asarray([1, 0], np.uint8)     # column head first: head order must not matter
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, 0.37)
    for b in range(2):
        for h in range(H):
            sets = brute_sets(rows[b], cols[b], P, int(hv[h]))
            Ob, Lb = brute_fwd(Q[b, h], K[b, h], V[b, h], sets, 0.37)
            np.testing.assert_allclose(O[b, h], Ob, rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(LSE[b, h], Lb, rtol=1e-12)


def test_zero_query_closed_form():
    # Q = 0  =>  O_k = mean of V over A_k, LSE_k = ln |A_k|: pins the set sizes exactly
    rows, cols, N = small_table(5, P=4, n_rows=4, n_cols=3, pad=3)
    H, d, P = 2, 5, 4
    _, K, V = rand_qkv(5, 1, H, N, d)
    Q = np.zeros_like(K)
    hv = np.asarray([0, 1], np.uint8)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, 1.0)
    for h in range(H):
        sets = brute_sets(rows[0], cols[0], P, int(hv[h]))
        for k in range(N):
            A = sorted(sets[k])
            if not A:
                assert np.all(O[0, h, k] == 0) and LSE[0, h, k] == -np.inf
                continue
            np.testing.assert_allclose(O[0, h, k], V[0, h, A].mean(axis=0), rtol=1e-13, atol=1e-15)
            assert abs(LSE[0, h, k] - math.log(len(A))) < 1e-13


def test_singleton_closed_form():
    # no prefix and all ids distinct: every token attends to itself only
    N, d = 7, 3
    rows = np.arange(1, N + 1, dtype=np.int32)[None]
    cols = np.arange(N, 0, -1, dtype=np.int32)[None]
    Q, K, V = rand_qkv(3, 1, 2, N, d)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, 0, np.asarray([0, 1], np.uint8), 0.5)
    np.testing.assert_allclose(O, V, rtol=1e-14)
    np.testing.assert_allclose(LSE, 0.5 * np.einsum("bhne,bhne->bhn", Q, K), rtol=1e-13)


def _sdpa(Q, K, V, valid, scale):
    """Library dense attention (torch CPU, fp64) restricted to valid keys, with autograd."""
    q, k, v = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    am = torch.tensor(valid, dtype=torch.bool)[None, None, None, :]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=am, scale=scale)
    return q, k, v, o


def test_one_row_spanning_table_is_dense_attention():
    # Section 3: when A holds all positions (except padding) we are in the dense case
    P, n_cols, pad = 3, 4, 2
    cells = [(1, c, 2) for c in range(1, n_cols + 1)]
    rows, cols = tables.custom_structure(P, cells, P + 2 * n_cols + pad)
    N = rows.shape[1]
    valid = rows[0] >= 0
    Q, K, V, dO = rand_qkv(11, 1, 1, N, 6, k=4)
    hv = np.asarray([0], np.uint8)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, 0.41)
    q, k, v, o = _sdpa(Q, K, V, valid, 0.41)
    np.testing.assert_allclose(O[..., valid, :], o.detach().numpy()[..., valid, :], rtol=1e-12, atol=1e-14)
    assert np.all(O[..., ~valid, :] == 0) and np.all(np.isneginf(LSE[..., ~valid]))
    s = 0.41 * torch.einsum("bhke,bhje->bhkj", q, k).detach()
    lse = torch.logsumexp(s[..., valid], dim=-1).numpy()
    np.testing.assert_allclose(LSE[..., valid], lse[..., valid], rtol=1e-12)
    # backward against the library's autograd; padding query rows carry no gradient
    dOm = dO.copy()
    dOm[..., ~valid, :] = 0
    o.backward(torch.tensor(dOm))
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, rows, cols, P, hv, 0.41)
    np.testing.assert_allclose(dQ, q.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dK, k.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dV, v.grad.numpy(), rtol=1e-10, atol=1e-13)
    assert np.all(dQ[..., ~valid, :] == 0) and np.all(dK[..., ~valid, :] == 0) and np.all(dV[..., ~valid, :] == 0)


def test_prefix_rows_do_not_depend_on_the_view():
    rows, cols, N = small_table(9, P=4)
    Q1, K1, V1 = rand_qkv(9, 1, 1, N, 4)
    Q, K, V = (np.repeat(x, 2, axis=1) for x in (Q1, K1, V1))
    O, LSE = oracle.fwd(Q, K, V, rows, cols, 4, np.asarray([0, 1], np.uint8), 0.5)
    np.testing.assert_array_equal(O[0, 0, :4], O[0, 1, :4])
    np.testing.assert_array_equal(LSE[0, 0, :4], LSE[0, 1, :4])
    assert not np.allclose(O[0, 0, 4:], O[0, 1, 4:])


# ---------------------------------------------------------------- equivariance

def test_permutation_and_relabelling_equivariance():
    rows, cols, N = small_table(21, P=3, n_rows=4, n_cols=3, pad=2)
    P, H, d = 3, 2, 4
    hv = np.asarray([0, 1], np.uint8)
    Q, K, V, dO = rand_qkv(21, 1, H, N, d, k=4)
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, 0.6)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, rows, cols, P, hv, 0.6)
    rng = np.random.default_rng(21)
    # permute the non-prefix positions (table tokens and padding travel with their ids)
    sigma = np.concatenate([np.arange(P), P + rng.permutation(N - P)])
    # relabel ids injectively (pattern has no positional or ordinal term)
    relabel_r = rng.permutation(20)[:6] + 1
    relabel_c = rng.permutation(20)[:5] + 1
    r2 = np.where(rows >= 1, relabel_r[np.maximum(rows, 0)], rows)[:, sigma].astype(np.int32)
    c2 = np.where(cols >= 1, relabel_c[np.maximum(cols, 0)], cols)[:, sigma].astype(np.int32)
    args = [x[:, :, sigma] for x in (Q, K, V, dO)]
    O2, LSE2 = oracle.fwd(args[0], args[1], args[2], r2, c2, P, hv, 0.6)
    dQ2, dK2, dV2 = oracle.bwd(*args, r2, c2, P, hv, 0.6)
    np.testing.assert_allclose(O2, O[:, :, sigma], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(LSE2, LSE[:, :, sigma], rtol=1e-12)
    for a, b in ((dQ2, dQ), (dK2, dK), (dV2, dV)):
        np.testing.assert_allclose(a, b[:, :, sigma], rtol=1e-10, atol=1e-13)


# ---------------------------------------------------------------- backward

def test_bwd_finite_differences():
    rows, cols, N = small_table(31, P=2, n_rows=2, n_cols=2, max_len=2, pad=1)
    P, H, d, scale = 2, 2, 3, 0.7
    hv = np.asarray([0, 1], np.uint8)
    Q, K, V, W = rand_qkv(31, 1, H, N, d, k=4)
    dQ, dK, dV = oracle.bwd(Q, K, V, W, rows, cols, P, hv, scale)

    def loss(q, k, v):
        O, _ = oracle.fwd(q, k, v, rows, cols, P, hv, scale)
        return float(np.sum(O * W))

    eps = 1e-6
    for name, X, G in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        num = np.zeros_like(X)
        it = np.nditer(X, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            Xp, Xm = X.copy(), X.copy()
            Xp[i] += eps
            Xm[i] -= eps
            a = [Q, K, V]
            a[["Q", "K", "V"].index(name)] = Xp
            lp = loss(*a)
            a[["Q", "K", "V"].index(name)] = Xm
            lm = loss(*a)
            num[i] = (lp - lm) / (2 * eps)
        np.testing.assert_allclose(G, num, rtol=2e-6, atol=2e-8, err_msg=name)


def test_bwd_against_autograd_of_masked_softmax():
    # independent derivation: torch autograd through a masked softmax built from the brute-force sets
    rows, cols, N = small_table(41, P=3, pad=2)
    P, H, d, scale = 3, 2, 4, 0.45
    hv = np.asarray([1, 0], np.uint8)
    Q, K, V, dO = rand_qkv(41, 1, H, N, d, k=4)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, rows, cols, P, hv, scale)
    q, k, v = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    M = np.zeros((1, H, N, N), dtype=bool)
    for h in range(H):
        for kk, A in enumerate(brute_sets(rows[0], cols[0], P, int(hv[h]))):
            M[0, h, kk, sorted(A)] = True
    Mt = torch.tensor(M)
    s = scale * torch.einsum("bhke,bhje->bhkj", q, k)
    s = s.masked_fill(~Mt, float("-inf"))
    rowvalid = Mt.any(-1, keepdim=True)
    p = torch.where(rowvalid, torch.softmax(torch.where(rowvalid, s, torch.zeros_like(s)), -1) * Mt, torch.zeros_like(s))
    o = torch.einsum("bhkj,bhje->bhke", p, v)
    o.backward(torch.tensor(dO))
    np.testing.assert_allclose(dQ, q.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dK, k.grad.numpy(), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dV, v.grad.numpy(), rtol=1e-10, atol=1e-13)
    # identities: sum_j dV_j = sum over valid k of dO_k (softmax rows sum to one)
    valid = rows[0] >= 0
    np.testing.assert_allclose(dV.sum(axis=2), dO[:, :, valid].sum(axis=2), rtol=1e-11)


def test_batched_calls_equal_per_example_calls():
    # The examples of a batch are independent (Section 3 defines the pattern per example): a call on
    # B = 3 examples with different structures must return, example by example, what three B = 1
    # calls return.  Pins the per-example offsets of every array inside the oracle's loops.
    rows, cols, N = small_table(51, P=3, n_rows=3, n_cols=2, max_len=3, pad=2, B=3)
    P, H, d, scale = 3, 3, 4, 0.8
    hv = np.asarray([0, 1, 0], np.uint8)
    Q, K, V, dO = rand_qkv(51, 3, H, N, d, k=4)
    assert not np.array_equal(rows[0], rows[1]) and not np.array_equal(rows[1], rows[2])
    O, LSE = oracle.fwd(Q, K, V, rows, cols, P, hv, scale)
    dQ, dK, dV = oracle.bwd(Q, K, V, dO, rows, cols, P, hv, scale)
    for b in range(3):
        s = slice(b, b + 1)
        O1, LSE1 = oracle.fwd(Q[s], K[s], V[s], rows[s], cols[s], P, hv, scale)
        g1 = oracle.bwd(Q[s], K[s], V[s], dO[s], rows[s], cols[s], P, hv, scale)
        assert np.array_equal(O[s], O1) and np.array_equal(LSE[s], LSE1)
        for a, b1 in zip((dQ, dK, dV), g1):
            assert np.array_equal(a[s], b1)


# ---------------------------------------------------------------- plan

def rank_formula(keys):
    """pos(k) = #{j : key_j < key_k} + #{j < k : key_j = key_k}   (O(N^2), unique stable order)."""
    N = len(keys)
    pos = [sum(1 for j in range(N) if keys[j] < keys[k]) + sum(1 for j in range(k) if keys[j] == keys[k])
           for k in range(N)]
    return pos


@pytest.mark.parametrize("name,seed", [("tiny", 1), ("bert", 2)])
def test_plan_against_rank_formula(name, seed):
    cfg = tables.CONFIGS[name]
    rows, cols, info = tables.make_structure(cfg, seed=seed)
    N = info["N"]
    rng = np.random.default_rng(seed)
    # shuffle the table part of example 0 so that the order is not already sorted
    sh = cfg.P + rng.permutation(N - cfg.P)
    rows[0, cfg.P:] = rows[0, sh]
    cols[0, cfg.P:] = cols[0, sh]
    for view, ids, max_id in ((0, rows, cfg.n_rows), (1, cols, cfg.n_cols)):
        perm, inv, seg = oracle.plan(rows, cols, cfg.P, view, max_id)
        for b in range(min(cfg.B, 2)):
            keys = [(0, 0) if k < cfg.P else ((1, int(ids[b, k])) if ids[b, k] >= 0 else (2, 0))
                    for k in range(N)]
            pos = rank_formula(keys)
            assert inv[b].tolist() == pos
            assert sorted(perm[b].tolist()) == list(range(N))
            assert np.array_equal(inv[b][perm[b]], np.arange(N))
            nv = int(np.sum(ids[b] >= 0))
            assert seg[b, 0] == cfg.P and seg[b, -1] == nv and np.all(np.diff(seg[b]) >= 0)
            for s in range(max_id + 1):
                members = perm[b, seg[b, s]:seg[b, s + 1]]
                assert np.all(ids[b, members] == s) and np.all(members >= cfg.P)
                assert np.all(np.diff(members) > 0)           # stable: original order kept
                assert len(members) == int(np.sum(ids[b, cfg.P:] == s))
            assert np.all(ids[b, perm[b, nv:]] < 0)


def test_row_major_table_column_view_is_column_traversal():
    # stable sort of a row-major table by column id visits column 1 top to bottom, then column 2, ...
    cells = [(r, c, 1) for r in (1, 2, 3) for c in (1, 2)]
    rows, cols = tables.custom_structure(1, cells)
    perm, _, seg = oracle.plan(rows, cols, 1, 1, 2)
    assert perm[0].tolist() == [0, 1, 3, 5, 2, 4, 6]
    assert seg[0].tolist() == [1, 1, 4, 7]
    perm_r, _, seg_r = oracle.plan(rows, cols, 1, 0, 3)
    assert perm_r[0].tolist() == list(range(7))
    assert seg_r[0].tolist() == [1, 1, 3, 5, 7]
