"""Fidelity diagnostics from the exact per-block logit statistics (ckv_exact_blocks; App. B of the paper).

The kernel reads every key and returns, per query head and block, logZ_b = log sum_j e^{z_j}, the mean logit and the
logit variance.  Everything here is block-level arithmetic on those arrays (numpy, float64): exact block masses, exact
compensation residuals, KL divergences of a selection, and rank agreement of the scorer with the exact residual.
Not part of the decode step.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Sequence

import numpy as np


@dataclass
class ExactUnit:
    """Exact quantities of one (sequence, KV head): arrays are [G][X]."""
    p: np.ndarray        # block mass Z_b / sum_c Z_c (Eq. 3)
    sigma2: np.ndarray   # within-block logit variance (what Eq. 8 estimates)
    rho: np.ndarray      # compensation residual p_b (1 - |b| e^{zmean_b} / Z_b) (App. B.1)
    logZ: np.ndarray     # log Z_b
    logW: np.ndarray     # log(|b| e^{zmean_b}): the mass mean compensation gives the block


def exact_unit(logZ, zmean, zvar, n_tokens: int, block_size: int) -> ExactUnit:
    """logZ, zmean, zvar: [G][>= X] rows of one unit as returned by ckv_exact_blocks."""
    x = -(-n_tokens // block_size)
    lz = np.asarray(logZ, np.float64)[:, :x]
    zm = np.asarray(zmean, np.float64)[:, :x]
    cnt = np.minimum(block_size, n_tokens - block_size * np.arange(x)).astype(np.float64)
    m = lz.max(axis=1, keepdims=True)
    z = np.exp(lz - m)
    p = z / z.sum(axis=1, keepdims=True)
    logw = np.log(cnt)[None, :] + zm
    rho = p * (1.0 - np.exp(np.minimum(logw - lz, 0.0)))   # |b| e^{zmean} <= Z_b (Jensen); the min guards rounding
    return ExactUnit(p=p, sigma2=np.asarray(zvar, np.float64)[:, :x], rho=rho, logZ=lz, logW=logw)


def kl_of_selection(e: ExactUnit, ids: Sequence[int], drop: bool = False) -> np.ndarray:
    """KL(P_hat || P) per head for the selected blocks `ids`: log(D / D_hat) with mean compensation (the
    log-partition gap of App. A.5), -log sum_{b in S} p_b when the other blocks are dropped."""
    g, x = e.logZ.shape
    sel = np.zeros(x, bool)
    sel[np.asarray(ids, int)] = True
    m = e.logZ.max(axis=1, keepdims=True)
    d_full = np.exp(e.logZ - m).sum(axis=1)
    d_hat = np.exp(e.logZ - m)[:, sel].sum(axis=1)
    if not drop:
        d_hat = d_hat + np.exp(e.logW - m)[:, ~sel].sum(axis=1)
    return np.log(d_full / d_hat)


def residual_capture(e: ExactUnit, ids: Sequence[int]) -> float:
    """Share of the group's total exact residual that lies in the selected blocks."""
    t = e.rho.sum(axis=0)
    return float(t[np.asarray(ids, int)].sum() / max(t.sum(), 1e-300))


def _ranks(a: np.ndarray) -> np.ndarray:
    order = np.argsort(a, kind="stable")
    r = np.empty(len(a), np.float64)
    r[order] = np.arange(len(a))
    # average the ranks of ties
    vals, inv, counts = np.unique(a, return_inverse=True, return_counts=True)
    sums = np.zeros(len(vals)); np.add.at(sums, inv, r)
    return sums[inv] / counts[inv]


def spearman(scores: np.ndarray, e: ExactUnit) -> float:
    """Rank correlation between the scorer's S_b and the exact group residual T_b = sum_g rho_{g,b}."""
    t = e.rho.sum(axis=0)
    s = np.asarray(scores, np.float64)[:len(t)]
    rs, rt = _ranks(s), _ranks(t)
    rs -= rs.mean(); rt -= rt.mean()
    den = np.sqrt((rs * rs).sum() * (rt * rt).sum())
    return float((rs * rt).sum() / den) if den > 0 else 0.0


def exact_topk(e: ExactUnit, k: int, sink: int = 1, recent: int = 2) -> np.ndarray:
    """The selection an exact-residual oracle would make under the same budget and mandatory blocks."""
    x = e.rho.shape[1]
    mand = [b for b in range(x) if b < sink or b >= x - recent]
    if k >= x:
        return np.arange(x)
    t = e.rho.sum(axis=0)
    rest = [b for b in np.argsort(-t, kind="stable") if b not in set(mand)]
    return np.array(sorted(mand + rest[:max(k - len(mand), 0)]))


def report(config: int = 2, units: int = 4) -> dict:
    """Runs one decode step of a synthetic configuration on cuda:0 and summarises the scorer's fidelity on a few
    units: rank agreement with the exact residual, residual captured by the selection (and by the exact-residual
    selection under the same budget), KL of the compensated and of the dropped approximation."""
    import torch

    from . import binding, synth
    w = synth.CONFIGS[config]
    k_pool, v_pool, table, lens = synth.make_pools(w)
    ckv = binding.CompKV(w.num_q_heads, w.num_kv_heads, w.batch, synth.pages_per_seq(w), k_pool.shape[0],
                         block_size=w.block_size, var_groups=w.var_groups)
    k_pool, v_pool, table, lens = (t.cuda() for t in (k_pool, v_pool, table, lens))
    n_max = int(lens.max())
    q = torch.from_numpy(synth.queries(w, 0)).bfloat16().cuda()
    ckv.stats_build(k_pool, v_pool, table, lens, n_max)
    out, lse, ids, cnt = ckv.decode(q, k_pool, v_pool, table, lens, n_max, w.budget_tokens)
    dense, _ = ckv.dense_decode(q, k_pool, v_pool, table, lens, n_max)
    scores = ckv.copy_scores(w.batch)
    logZ, zmean, zvar = ckv.exact_blocks(q, k_pool, table, lens, n_max)
    torch.cuda.synchronize()
    G, bs, k = w.group, w.block_size, w.budget_tokens // w.block_size
    rows = []
    for u in range(min(units, w.batch * w.num_kv_heads)):
        s, h = divmod(u, w.num_kv_heads)
        n = int(lens[s])
        hs = slice(h * G, (h + 1) * G)
        e = exact_unit(logZ[s, hs].cpu().numpy(), zmean[s, hs].cpu().numpy(), zvar[s, hs].cpu().numpy(), n, bs)
        sel = ids[s, h, :int(cnt[s, h])].cpu().numpy()
        best = exact_topk(e, k)
        o, dn = out[s, hs].double().cpu().numpy(), dense[s, hs].double().cpu().numpy()
        rows.append({"unit": (s, h), "spearman": spearman(scores[s, h].cpu().numpy(), e),
                     "residual_capture": residual_capture(e, sel), "residual_capture_exact_topk": residual_capture(e, best),
                     "kl_mean": float(kl_of_selection(e, sel).mean()), "kl_drop": float(kl_of_selection(e, sel, True).mean()),
                     "kl_mean_exact_topk": float(kl_of_selection(e, best).mean()),
                     "out_vs_dense": float(np.abs(o - dn).max() / np.abs(dn).max())})
    return {"config": w.name, "rows": rows}


if __name__ == "__main__":
    import json
    import sys
    print(json.dumps(report(int(sys.argv[1]) if len(sys.argv) > 1 else 2), indent=1))
