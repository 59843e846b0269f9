"""Seeded synthetic inputs for the CompKV decode path.

This module only draws random numbers and arranges them into the shapes the
decode path consumes (queries, per-unit K/V, page tables, paged pools).  It holds
none of the method's arithmetic: no statistics, scores, selection or attention.
Both the CPU oracle's tests and the CUDA path's tests/bench take their inputs
from here, so the two sides always see identical values.

Value recipe (one "unit" = one sequence x one KV head):
  * keys of every 16-token unit: centre c ~ N(0,1)^d plus per-token noise
    s * eps, eps ~ N(0,I), with s drawn per 16-token unit from {0.05, 0.3, 1.0};
  * optional outlier channels: `outlier_dims` coordinates per unit whose key
    entries (centre and noise) are multiplied by `outlier_scale`;
  * optional needles: `needles` token positions per unit, outside the first
    block and the last two blocks of the prefilled cache, whose keys get
    + (6 sqrt(d) / |qbar|^2) * qbar added, qbar being the mean step-0 query of
    the unit's GQA group (so the group-mean logit of a needle rises by 6);
  * values ~ N(0,1)^d, queries ~ N(0,1)^d, step-t query = step-0 query + 0.3 N(0,I);
  * everything is rounded once to bf16 (round-to-nearest-even) and handed out as
    float32 holding exactly those bf16 values.

The random streams are counter-based (Philox) and keyed by
(seed, tensor id, sequence, head), so any unit can be regenerated on its own.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

_T_Q, _T_KEYS, _T_VALS, _T_META, _T_LEN, _T_PAGES, _T_QSTEP = 1, 2, 3, 4, 5, 6, 7
NOISE_LEVELS = np.array([0.05, 0.3, 1.0], dtype=np.float32)
MIX_UNIT = 16  # centres / noise levels are drawn per 16 tokens whatever the block size


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    ctx: int                      # prefilled tokens per sequence (upper bound when ragged)
    budget_tokens: int
    seed: int
    ctx_min: Optional[int] = None  # ragged: lengths uniform in [ctx_min, ctx]
    head_dim: int = 128
    block_size: int = 16
    page_size: int = 16
    var_groups: int = 4
    needles: int = 0
    outlier_dims: int = 0
    outlier_scale: float = 8.0
    decode_steps: int = 1          # tokens appended after the prefill
    shuffle_pages: bool = True

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_BASE_SEED = 260926300

CONFIGS: Dict[int, Workload] = {
    1: Workload("toy_4k", batch=1, num_q_heads=4, num_kv_heads=1, ctx=4096, budget_tokens=256,
                seed=_BASE_SEED + 1, needles=8),
    2: Workload("llama8b_32k", batch=1, num_q_heads=32, num_kv_heads=8, ctx=32768, budget_tokens=1024,
                seed=_BASE_SEED + 2, needles=64, outlier_dims=4),
    3: Workload("llama8b_128k_b4", batch=4, num_q_heads=32, num_kv_heads=8, ctx=131072, budget_tokens=2048,
                seed=_BASE_SEED + 3, needles=64, outlier_dims=4, decode_steps=64),
    4: Workload("qwen32b_ragged_b16", batch=16, num_q_heads=64, num_kv_heads=8, ctx=65536, ctx_min=16384,
                budget_tokens=1024, seed=_BASE_SEED + 4, needles=64, outlier_dims=4),
    5: Workload("llama8b_128k_sweep", batch=1, num_q_heads=32, num_kv_heads=8, ctx=131072, budget_tokens=2048,
                seed=_BASE_SEED + 5, needles=64, outlier_dims=4),
}
SWEEP_BLOCK_SIZES = (16, 32, 64)
SWEEP_BUDGETS = (512, 1024, 2048, 4096)


def _rng(seed: int, tensor: int, s: int = 0, h: int = 0, extra: int = 0) -> np.random.Generator:
    key1 = (tensor << 56) | (extra << 40) | (s << 20) | h
    return np.random.Generator(np.random.Philox(key=[seed, key1]))


def round_bf16_(x: np.ndarray) -> np.ndarray:
    """Round a float32 array in place to the nearest bf16 value (ties to even)."""
    assert x.dtype == np.float32 and x.flags.c_contiguous
    u = x.reshape(-1).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    u += bias
    u &= np.uint32(0xFFFF0000)
    return x


def seq_lens(w: Workload) -> np.ndarray:
    """Prefilled length of every sequence, int32 [batch]."""
    if w.ctx_min is None:
        return np.full(w.batch, w.ctx, dtype=np.int32)
    g = _rng(w.seed, _T_LEN)
    return g.integers(w.ctx_min, w.ctx + 1, size=w.batch).astype(np.int32)


def queries(w: Workload, step: int = 0) -> np.ndarray:
    """Decode queries of one step, float32 [batch][num_q_heads][head_dim] (bf16 values)."""
    q0 = _rng(w.seed, _T_Q).standard_normal((w.batch, w.num_q_heads, w.head_dim), dtype=np.float32)
    if step > 0:
        q0 = q0 + np.float32(0.3) * _rng(w.seed, _T_QSTEP, extra=step).standard_normal(q0.shape, dtype=np.float32)
    q0 = np.ascontiguousarray(q0, dtype=np.float32)
    return round_bf16_(q0)


def _step0_group_mean_query(w: Workload, s: int, h: int) -> np.ndarray:
    q = queries(w, 0)[s, h * w.group:(h + 1) * w.group]
    return q.mean(axis=0, dtype=np.float64)


def needle_positions(w: Workload, s: int, h: int, n_prefill: int) -> np.ndarray:
    """Token positions of the planted needles of one unit (sorted, distinct)."""
    if w.needles == 0:
        return np.zeros(0, dtype=np.int64)
    bs = w.block_size
    x = -(-n_prefill // bs)
    lo, hi = bs, (x - 2) * bs  # outside block 0 and blocks X-1, X-2
    if hi - lo < w.needles:
        return np.zeros(0, dtype=np.int64)
    g = _rng(w.seed, _T_META, s, h, extra=1)
    return np.sort(g.choice(hi - lo, size=w.needles, replace=False) + lo).astype(np.int64)


def outlier_channels(w: Workload, s: int, h: int) -> np.ndarray:
    if w.outlier_dims == 0:
        return np.zeros(0, dtype=np.int64)
    g = _rng(w.seed, _T_META, s, h, extra=2)
    return np.sort(g.choice(w.head_dim, size=w.outlier_dims, replace=False)).astype(np.int64)


def _mixture(w: Workload, s: int, h: int, n_prefill: int):
    """Centres and noise levels of every 16-token unit of one (sequence, KV head), and the key stream."""
    n_units = -(-(n_prefill + w.decode_steps) // MIX_UNIT)
    gk = _rng(w.seed, _T_KEYS, s, h)
    centres = gk.standard_normal((n_units, w.head_dim), dtype=np.float32)
    levels = NOISE_LEVELS[gk.integers(0, 3, size=n_units)]
    return centres, levels, gk


def _finish_keys(w: Workload, s: int, h: int, k: np.ndarray, first_row: int, n_prefill: int) -> np.ndarray:
    ch = outlier_channels(w, s, h)
    if ch.size:
        k[:, ch] *= np.float32(w.outlier_scale)
    pos = needle_positions(w, s, h, n_prefill) - first_row
    pos = pos[(pos >= 0) & (pos < k.shape[0])]
    if pos.size:
        qbar = _step0_group_mean_query(w, s, h)
        bump = (6.0 * np.sqrt(w.head_dim) / float(qbar @ qbar)) * qbar
        k[pos] += bump.astype(np.float32)[None, :]
    return round_bf16_(np.ascontiguousarray(k))


def unit_tail(w: Workload, s: int, h: int) -> Tuple[np.ndarray, np.ndarray]:
    """Rows the decode steps append to one unit, float32 [decode_steps][head_dim] each.

    They continue the block mixture (same centre while inside the 16-token unit
    the prefill ended in, a new centre and noise level at each 16-token boundary)
    and come from random streams of their own, so they cost nothing to regenerate.
    """
    d = w.head_dim
    n_prefill = int(seq_lens(w)[s])
    centres, levels, _ = _mixture(w, s, h, n_prefill)
    rows = np.arange(n_prefill, n_prefill + w.decode_steps)
    u = rows // MIX_UNIT
    k = _rng(w.seed, _T_KEYS, s, h, extra=1).standard_normal((w.decode_steps, d), dtype=np.float32)
    k *= levels[u][:, None]
    k += centres[u]
    k = _finish_keys(w, s, h, k, n_prefill, n_prefill)
    v = _rng(w.seed, _T_VALS, s, h, extra=1).standard_normal((w.decode_steps, d), dtype=np.float32)
    return k, round_bf16_(np.ascontiguousarray(v))


def unit_kv(w: Workload, s: int, h: int, with_tail: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """Keys and values of one (sequence, KV head): float32 [n][head_dim] each (bf16 values).

    n = prefill length (+ decode_steps with with_tail: the rows past the prefill
    are the tokens the decode steps append, in order).
    """
    d = w.head_dim
    n_prefill = int(seq_lens(w)[s])
    centres, levels, gk = _mixture(w, s, h, n_prefill)
    nu = -(-n_prefill // MIX_UNIT)
    k = gk.standard_normal((nu, MIX_UNIT, d), dtype=np.float32)
    k *= levels[:nu, None, None]
    k += centres[:nu, None, :]
    k = _finish_keys(w, s, h, k.reshape(nu * MIX_UNIT, d)[:n_prefill], 0, n_prefill)
    v = _rng(w.seed, _T_VALS, s, h).standard_normal((n_prefill, d), dtype=np.float32)
    v = round_bf16_(np.ascontiguousarray(v))
    if with_tail and w.decode_steps > 0:
        kt, vt = unit_tail(w, s, h)
        k = np.concatenate([k, kt])
        v = np.concatenate([v, vt])
    return k, v


def pages_per_seq(w: Workload) -> int:
    """Row stride of the page table: pages that hold ctx + decode_steps tokens."""
    cap = w.ctx + w.decode_steps
    per_block = w.block_size // w.page_size
    blocks = -(-cap // w.block_size)
    return blocks * per_block


def page_table(w: Workload) -> Tuple[np.ndarray, int]:
    """int32 [batch][pages_per_seq] physical page of every logical page, and the pool size.

    Every sequence owns pages for its prefill plus the tokens the decode steps
    append; unused table slots hold -1.  With shuffle_pages the pool order is a
    seeded random permutation, so logically adjacent pages are not adjacent in memory.
    """
    lens = seq_lens(w).astype(np.int64) + w.decode_steps
    need = -(-lens // w.page_size)
    total = int(need.sum())
    perm = np.arange(total, dtype=np.int64)
    if w.shuffle_pages:
        perm = _rng(w.seed, _T_PAGES).permutation(total)
    table = np.full((w.batch, pages_per_seq(w)), -1, dtype=np.int32)
    off = 0
    for s in range(w.batch):
        table[s, :need[s]] = perm[off:off + need[s]]
        off += int(need[s])
    return table, total


def fill_pools(w: Workload, k_pool, v_pool, table: np.ndarray, units: Optional[List[Tuple[int, int]]] = None,
               threads: int = 8) -> None:
    """Scatter every unit's K/V rows into the paged pools.

    k_pool / v_pool: CPU torch tensors [num_pages][num_kv_heads][page_size][head_dim]
    (bf16 or float32).  Rows of a sequence past its last token stay as they were.
    """
    import torch
    from concurrent.futures import ThreadPoolExecutor

    ps, d = w.page_size, w.head_dim
    todo = units if units is not None else [(s, h) for s in range(w.batch) for h in range(w.num_kv_heads)]

    def one(sh):
        s, h = sh
        k, v = unit_kv(w, s, h)
        n = k.shape[0]
        n_pages = -(-n // ps)
        pad = n_pages * ps - n
        if pad:
            k = np.concatenate([k, np.zeros((pad, d), np.float32)])
            v = np.concatenate([v, np.zeros((pad, d), np.float32)])
        idx = torch.from_numpy(table[s, :n_pages].astype(np.int64))
        k_pool[idx, h] = torch.from_numpy(k).view(n_pages, ps, d).to(k_pool.dtype)
        v_pool[idx, h] = torch.from_numpy(v).view(n_pages, ps, d).to(v_pool.dtype)

    if threads > 1 and len(todo) > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(one, todo))
    else:
        for sh in todo:
            one(sh)


def make_pools(w: Workload, dtype=None, units: Optional[List[Tuple[int, int]]] = None, threads: int = 8):
    """Allocate CPU pools, fill them, and return (k_pool, v_pool, page_table int32 tensor, seq_lens int32 tensor).

    The rows of the tokens the decode steps append are already in the pools (a
    decode step re-writes the same values), which lets a test compare
    build-then-append with a build over the longer cache.
    """
    import torch
    dtype = dtype or torch.bfloat16
    table, total = page_table(w)
    shape = (total, w.num_kv_heads, w.page_size, w.head_dim)
    k_pool = torch.zeros(shape, dtype=dtype)
    v_pool = torch.zeros(shape, dtype=dtype)
    fill_pools(w, k_pool, v_pool, table, units=units, threads=threads)
    return k_pool, v_pool, torch.from_numpy(table), torch.from_numpy(seq_lens(w))


def appended_rows(w: Workload, step: int) -> Tuple[np.ndarray, np.ndarray]:
    """K and V rows that decode step `step` appends: float32 [batch][num_kv_heads][head_dim] each."""
    k_new = np.zeros((w.batch, w.num_kv_heads, w.head_dim), np.float32)
    v_new = np.zeros_like(k_new)
    for s in range(w.batch):
        for h in range(w.num_kv_heads):
            k, v = unit_tail(w, s, h)
            k_new[s, h] = k[step]
            v_new[s, h] = v[step]
    return k_new, v_new
