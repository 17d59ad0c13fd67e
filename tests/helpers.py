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


def view_positions(rows, cols, P, head_view):
    """int64 [B, H, N]: position of every token in the stable order of its head's view (prefix first,
    then the table tokens by id and original position, padding last).  Plain numpy sort; used only
    to shape test inputs."""
    B, N = rows.shape
    out = np.empty((B, len(head_view), N), np.int64)
    for b in range(B):
        for h, v in enumerate(head_view):
            ids = (rows if v == 0 else cols)[b].astype(np.int64)
            cls = np.where(np.arange(N) < P, 0, np.where(ids >= 0, 1, 2))
            key = cls * (1 << 40) + np.where(cls == 1, ids, 0) * (1 << 20) + np.arange(N)
            order = np.argsort(key, kind="stable")
            out[b, h, order] = np.arange(N)
    return out


def ramp_case(cfg, rows, cols, vals, growth_log2, scale, q_mean=1.0):
    """Shapes the values of a case so that the scaled scores of every query grow along the order in
    which its head visits the keys, by about `growth_log2` powers of two per 128 keys: every
    component of Q gets the mean `q_mean` and every component of K a ramp over the key's position in
    the head's view.  Returns new bf16-exact arrays (Q, K changed; V, dO kept)."""
    hv = tables.head_view(cfg)
    pos = view_positions(rows, cols, cfg.P, hv).astype(np.float64)            # [B, H, N]
    slope = growth_log2 * np.log(2.0) / (scale * cfg.d * q_mean * 128.0)
    out = dict(vals)
    out["Q"] = tables.round_to_bf16((vals["Q"] + q_mean).astype(np.float32))
    out["K"] = tables.round_to_bf16((vals["K"] + (slope * pos)[..., None]).astype(np.float32))
    return out
