"""Seeded synthetic table workloads for multi-view attention.

This module only draws random structure (row/column ids) and random values.
It holds none of the attention arithmetic, so both the CPU oracle's tests and
the CUDA library's tests and benchmark may use it.

Token sequence layout (paper Section 3): a prefix of `P` query/text tokens
(row id = column id = 0) followed by the table flattened in row-major order,
rows and columns numbered from 1.  Every cell contributes `len` consecutive
tokens carrying that cell's (row, column).  A table longer than `N - P` tokens
is cut at `N` (trailing rows dropped, the last cell possibly partial); a
shorter one is followed by padding tokens whose ids are -1.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class TableConfig:
    name: str
    B: int
    H: int
    n_row_heads: int          # heads [0, n_row_heads) use the row view, the rest the column view
    d: int
    N: Optional[int]          # padded sequence length; None = no padding (N = P + table tokens)
    P: int                    # prefix length |Q|
    n_rows: int
    n_cols: int
    cell_law: str             # "uniform" | "geometric" | "zipf"
    cell_param: float         # uniform: max length; geometric: p; zipf: s
    cell_cap: int
    dtype: str                # "f32" | "bf16"
    value_scale: float
    merged_row_frac: float = 0.0
    backward: bool = True


CONFIGS: Dict[str, TableConfig] = {
    # B=1, H=4 (2 row + 2 column heads), d=16, fp32, 8 prefix tokens + 4x3 table, len U{1..4}
    "tiny": TableConfig("tiny", 1, 4, 2, 16, None, 8, 4, 3, "uniform", 4, 4, "f32", 1.0,
                        backward=False),
    # BERT-base layer shape
    "bert": TableConfig("bert", 8, 12, 6, 64, 512, 64, 16, 8, "geometric", 0.5, 8, "bf16", 0.5),
    # medium table
    "medium": TableConfig("medium", 4, 12, 6, 64, 2048, 128, 64, 10, "geometric", 0.4, 12,
                          "bf16", 0.5),
    # long-document headline
    "long": TableConfig("long", 1, 12, 6, 64, 8192, 256, 400, 8, "geometric", 0.45, 16,
                        "bf16", 0.5),
    # skewed-structure stress
    "skew": TableConfig("skew", 2, 16, 8, 64, 4096, 128, 120, 30, "zipf", 1.2, 64, "bf16", 0.5,
                        merged_row_frac=0.10),
}


def head_view(cfg: TableConfig) -> np.ndarray:
    """uint8 [H]: 0 = row head, 1 = column head (row heads first)."""
    hv = np.ones(cfg.H, dtype=np.uint8)
    hv[: cfg.n_row_heads] = 0
    return hv


def _cell_lengths(cfg: TableConfig, rng: np.random.Generator, n: int) -> np.ndarray:
    if cfg.cell_law == "uniform":
        return rng.integers(1, int(cfg.cell_param) + 1, size=n)
    if cfg.cell_law == "geometric":
        # 1 + (failures before the first success) has support 1, 2, ...: numpy's geometric law
        return np.minimum(rng.geometric(cfg.cell_param, size=n), cfg.cell_cap)
    if cfg.cell_law == "zipf":
        k = np.arange(1, cfg.cell_cap + 1, dtype=np.float64)
        pmf = k ** (-cfg.cell_param)
        pmf /= pmf.sum()
        return rng.choice(np.arange(1, cfg.cell_cap + 1), size=n, p=pmf)
    raise ValueError(cfg.cell_law)


def make_structure(cfg: TableConfig, seed: int = 1234) -> Tuple[np.ndarray, np.ndarray, dict]:
    """Return (row_ids, col_ids) int32 [B, N] and a dict of realised statistics."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    per_example = []
    for _ in range(cfg.B):
        rows, cols = [], []
        merged = rng.random(cfg.n_rows) < cfg.merged_row_frac
        for r in range(1, cfg.n_rows + 1):
            if merged[r - 1]:
                # one cell spanning the whole row; it carries the first column's id
                ln = int(_cell_lengths(cfg, rng, 1)[0])
                rows += [r] * ln
                cols += [1] * ln
                continue
            lens = _cell_lengths(cfg, rng, cfg.n_cols)
            for c in range(1, cfg.n_cols + 1):
                ln = int(lens[c - 1])
                rows += [r] * ln
                cols += [c] * ln
        per_example.append((np.asarray(rows, np.int32), np.asarray(cols, np.int32)))

    if cfg.N is None:
        assert cfg.B == 1, "unpadded configs hold one example"
        N = cfg.P + len(per_example[0][0])
    else:
        N = cfg.N
    row_ids = np.full((cfg.B, N), -1, dtype=np.int32)
    col_ids = np.full((cfg.B, N), -1, dtype=np.int32)
    n_valid, rows_kept = [], []
    for b, (r, c) in enumerate(per_example):
        t = min(len(r), N - cfg.P)
        row_ids[b, : cfg.P] = 0
        col_ids[b, : cfg.P] = 0
        row_ids[b, cfg.P: cfg.P + t] = r[:t]
        col_ids[b, cfg.P: cfg.P + t] = c[:t]
        n_valid.append(cfg.P + t)
        rows_kept.append(int(r[t - 1]) if t > 0 else 0)
    info = {"N": N, "n_valid": n_valid, "rows_kept": rows_kept,
            "max_row_id": cfg.n_rows, "max_col_id": cfg.n_cols}
    return row_ids, col_ids, info


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32)


def make_values(cfg: TableConfig, N: int, seed: int = 5678,
                names=("Q", "K", "V", "dO")) -> Dict[str, np.ndarray]:
    """iid N(0,1)*value_scale float32 [B,H,N,d]; rounded to bf16-representable values for bf16
    configs.  Padding positions keep their (finite) random values so that leaks show up."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    out = {}
    for nm in names:
        x = rng.standard_normal((cfg.B, cfg.H, N, cfg.d), dtype=np.float32) * np.float32(cfg.value_scale)
        if cfg.dtype == "bf16":
            x = round_to_bf16(x)
        out[nm] = x
    return out


def custom_structure(P: int, cells, N: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Build ids for one example from an explicit list of (row, col, length) cells."""
    rows = [0] * P
    cols = [0] * P
    for r, c, ln in cells:
        rows += [r] * ln
        cols += [c] * ln
    n = len(rows)
    if N is None:
        N = n
    assert N >= n
    rows += [-1] * (N - n)
    cols += [-1] * (N - n)
    return (np.asarray(rows, np.int32)[None, :], np.asarray(cols, np.int32)[None, :])
