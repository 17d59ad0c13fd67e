"""Shared helpers of the GPU parity tests (no method arithmetic: data movement and comparisons)."""
import numpy as np
import torch

from workloads import tables

BF16_ATOL, BF16_RTOL = 2e-2, 1e-2     # |x - ref| <= atol + rtol * |ref| for bf16 tensors
F32_ATOL, F32_RTOL = 1e-5, 1e-5       # fp32 debug path


def tol(dtype):
    return (BF16_ATOL, BF16_RTOL) if dtype == "bf16" else (F32_ATOL, F32_RTOL)


def to_dev(x, dtype):
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t.float()


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def assert_close(got, ref, atol, rtol, what):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, what
    assert np.all(np.isfinite(got)), "%s: non-finite values" % what
    err = np.abs(got - ref)
    bound = atol + rtol * np.abs(ref)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError("%s: %d of %d elements out of tolerance; worst at %s: got %r ref %r "
                             "(max abs err %.3e)" % (what, int(bad.sum()), bad.size, i, got[i], ref[i],
                                                    err.max()))


def make_case(name, seed_structure=1234, seed_values=5678, shuffle=False):
    """Structure + values of a named config.  `shuffle` permutes the table tokens of every example
    (ids travel with the tokens), so that neither view is already in sorted order."""
    cfg = tables.CONFIGS[name]
    rows, cols, info = tables.make_structure(cfg, seed_structure)
    if shuffle:
        rng = np.random.default_rng(seed_structure + 99)
        for b in range(cfg.B):
            nv = info["n_valid"][b]
            sh = cfg.P + rng.permutation(nv - cfg.P)
            rows[b, cfg.P:nv] = rows[b, sh]
            cols[b, cfg.P:nv] = cols[b, sh]
    vals = tables.make_values(cfg, info["N"], seed_values)
    return cfg, rows, cols, info, vals
