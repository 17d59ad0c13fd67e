"""mate_cell_mean (per-cell mean of token logits, Section 4.1) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from workloads import tables

pytestmark = pytest.mark.gpu


def check(rows, cols, P, max_row, max_col, seed):
    import paper_2109_04312_b200 as m
    rng = np.random.default_rng(seed)
    logits = rng.standard_normal(rows.shape).astype(np.float32)
    r, c = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    plan = m.mate_plan(r, c, P, [0, 1], max_row, max_col)
    mean, count = m.mate_cell_mean(plan, torch.from_numpy(logits).cuda(), c)
    torch.cuda.synchronize()
    want_mean, want_count = oracle.cell_mean(logits, rows, cols, P, max_row, max_col)
    assert np.array_equal(count.cpu().numpy(), want_count)            # integer work: bit exact
    np.testing.assert_allclose(mean.cpu().numpy(), want_mean, rtol=1e-5, atol=1e-6)
    # without the counts
    mean2, none = m.mate_cell_mean(plan, torch.from_numpy(logits).cuda(), c, want_count=False)
    assert none is None and torch.equal(mean, mean2)                 # same result on every launch
    plan.destroy()


@pytest.mark.parametrize("name", ["tiny", "bert", "long", "skew"])
@pytest.mark.parametrize("shuffle", [False, True])
def test_cell_mean_on_the_workloads(name, shuffle):
    cfg, rows, cols, info, _ = hp.make_case(name, shuffle=shuffle)
    check(rows, cols, cfg.P, cfg.n_rows, cfg.n_cols, 3)


def test_cell_mean_edge_cases():
    # header row numbered 0, a column id above 128 (several passes over the columns), empty rows, no prefix
    rows, cols = tables.custom_structure(0, [(0, 1, 3), (0, 200, 2), (5, 1, 1), (5, 130, 40), (7, 0, 1)], 60)
    check(rows, cols, 0, 9, 200, 1)
    # only a prefix: every cell is empty
    z = np.zeros((2, 19), np.int32)
    check(z, z.copy(), 19, 3, 2, 2)
