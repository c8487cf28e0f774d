"""Shared helpers for the parity tests: the error metric, tolerances, tensor
plumbing between torch (GPU side) and numpy (oracle side), and compaction of a
paged KV cache to a few sampled sequences so the oracle can check full-size
workloads row by row."""
from __future__ import annotations

import numpy as np
import torch

from paper_2608_01891_b200 import inputs as IN

# Tolerances (max relative error per row, see row_rel_err) on bf16 inputs.
TOL_ATTN = 1e-2
TOL_FFN = 2e-2
TOL_GATE = 1e-6
TOL_LSE = 1e-3


def row_rel_err(got, want) -> float:
    """max over rows r of  max_i |got[r,i] - want[r,i]| / max(max_i |want[r,i]|, 1e-30).
    A row is the last dimension (one head's D-vector, one token's H-vector)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if not np.isfinite(got).all():
        return float("inf")
    num = np.abs(got - want).max(axis=-1)
    den = np.maximum(np.abs(want).max(axis=-1), 1e-30)
    return float((num / den).max())


def u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device) -> uint16 bit patterns on the host."""
    return IN.bf16_bits(t.detach().cpu().contiguous())


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def compact_kv(k_cache: torch.Tensor, v_cache: torch.Tensor, page_table, seq_lens, rows):
    """Gather the pages of the sampled sequences `rows` into a small host-side pool.
    Returns (k u16, v u16, table i32, lens i32) for the oracle; page ids are renumbered."""
    table = np.asarray(page_table)
    lens = np.asarray(seq_lens)
    new_rows, ids, o = [], [], 0
    max_pages = max((int(lens[b]) + 15) // 16 for b in rows)
    for b in rows:
        n = (int(lens[b]) + 15) // 16
        ids.extend(table[b, :n].tolist())
        r = np.zeros(max_pages, dtype=np.int32)
        r[:n] = np.arange(o, o + n)
        new_rows.append(r)
        o += n
    sel = torch.as_tensor(np.asarray(ids, dtype=np.int64), device=k_cache.device)
    k = u16(k_cache.index_select(0, sel))
    v = u16(v_cache.index_select(0, sel))
    return k, v, np.stack(new_rows), lens[list(rows)].astype(np.int32)
