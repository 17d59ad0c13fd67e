"""Parity of the forward's running-max bookkeeping against the oracle.

The tensor-core forward keeps one running row maximum per unit and re-bases it (scaling the
accumulated output) only when a key tile raises it by more than a threshold.  Random N(0,1)/2 inputs
never do that, so these cases shape the inputs: scores that grow along the order in which a head
visits its keys (slowly: below the threshold per tile, so the stale maximum is used and P exceeds 1;
moderately: every other tile re-bases; fast: every tile re-bases), on table-row units, on long
prefix units and on the split prefix units of the 8192-token workload, plus inputs with large random
scores.  Expected values are the fp64 oracle's (Section 3 head formula), tolerance as everywhere.

The shaped (ramp) cases check the forward only, which is where the bookkeeping under test lives.
Their keys have a large common component, and the backward takes D = rowsum(dO o O) from the bf16
output it is given: the rounding of O shifts dS of a whole row by a common amount, which a key
vector with a non-zero mean turns into an error of dQ and dK of scale * |mean K| * 2^-9 * |dO.O| --
a property of the bf16 interface, present in the SIMT kernels as well, and above the fixed absolute
tolerance for these inputs.  The large-random-score cases (zero-mean keys) check the backward too,
with dO scaled by a power of two that brings dQ back to its usual size (run_case(unit_grads=True):
exact, the backward is linear in dO)."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as hp
from tests.test_gpu_parity import custom_case, impls_for, mate, run_case
from workloads import tables

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,growth", [("medium", 5.0), ("medium", 12.0), ("medium", 40.0),
                                         ("skew", 9.0), ("long", 12.0), ("long", 3.0)])
def test_scores_growing_along_the_view_order(name, growth):
    cfg, rows, cols, info, vals = hp.make_case(name)
    scale = 1.0
    vals = hp.ramp_case(cfg, rows, cols, vals, growth, scale)
    run_case(cfg, rows, cols, vals, mate().IMPL_TCGEN05, backward=False, scale=scale)


@pytest.mark.parametrize("growth", [-12.0, -40.0])
def test_scores_falling_along_the_view_order(growth):
    # the first tile holds the maximum: later tiles contribute almost nothing and must not disturb it
    cfg, rows, cols, info, vals = hp.make_case("medium")
    vals = hp.ramp_case(cfg, rows, cols, vals, growth, 1.0)
    run_case(cfg, rows, cols, vals, mate().IMPL_TCGEN05, backward=False, scale=1.0)


def test_long_segments_with_growing_scores():
    # table-row units of many tiles: one column of 900 tokens and one row of 700
    cells = [(1, 1, 300), (2, 1, 300), (3, 1, 300), (4, 2, 700), (4, 3, 20)]
    cfg, rows, cols, vals = custom_case(40, cells, 40 + 1620 + 13, H=4)
    for growth in (6.0, 20.0):
        v = hp.ramp_case(cfg, rows, cols, vals, growth, 1.0)
        run_case(cfg, rows, cols, v, mate().IMPL_TCGEN05, backward=False, scale=1.0)


@pytest.mark.parametrize("value_scale,scale", [(2.0, 0.125), (1.0, 1.0), (3.0, 0.125)])
def test_large_random_scores(value_scale, scale):
    # scaled scores with a standard deviation of 4 to 8 (natural units): the tile maxima jump up and
    # down by many powers of two from tile to tile, the softmax is close to one-hot
    cfg0 = tables.CONFIGS["medium"]
    cfg = tables.TableConfig(**{**cfg0.__dict__, "value_scale": value_scale})
    rows, cols, info = tables.make_structure(cfg, 1234)
    vals = tables.make_values(cfg, info["N"], 77)
    for impl in impls_for(cfg):
        run_case(cfg, rows, cols, vals, impl, backward=(value_scale < 3.0), scale=scale, unit_grads=True)
