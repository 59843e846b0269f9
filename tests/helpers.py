"""Shared plumbing of the GPU parity tests: device setup from the seeded generator, oracle runs on
sampled units, and the comparison rules (tolerances stated here, used everywhere)."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import compkv_oracle as O
from paper_2609_26300_b200 import synth

# ---- tolerances (bf16 storage + fp32 accumulation vs the fp64 oracle) -------------------------------------
OUT_TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}   # max over heads of |o - o_ref|_inf / |o_ref|_inf
SCORE_RTOL = 1e-4        # block scores, where S_b >= 1e-30 * max S
TIE_RTOL = 1e-4          # selected ids may differ only on blocks whose score is this close to the threshold
STATS_RTOL = 1e-5        # summaries: |x - ref| <= STATS_RTOL * (|ref| + scale of the block's data)
LSE_ATOL = {torch.bfloat16: 1e-4, torch.float32: 1e-4}   # fp32 log-sum-exp on both layouts
# bf16 summaries (ckv_layout.stat_bf16): the oracle rounds its fp64 means to bf16 itself; where the GPU's fp32 mean
# falls on the other side of a rounding boundary (about 1 block in 100 has such a coordinate) one coordinate of the
# mean key differs by a bf16 ulp, which moves that block's logit by ~1e-2 relative
SCORE_RTOL_STAT_BF16 = 5e-2
LSE_ATOL_STAT_BF16 = 2e-3


@dataclass
class Device:
    w: synth.Workload
    ckv: object
    k_pool: torch.Tensor
    v_pool: torch.Tensor
    table: torch.Tensor
    lens: torch.Tensor
    max_len: int
    dtype: torch.dtype


def setup(w: synth.Workload, kv_dtype: torch.dtype = torch.bfloat16, poison_tail: bool = True,
          var_groups: Optional[int] = None, group_layout: int = 1, sink: int = 1, recent: int = 2,
          sm_scale: float = 0.0, variant: int = 0, stat_bf16: int = 0) -> Device:
    from paper_2609_26300_b200 import binding
    k_pool, v_pool, table, lens = synth.make_pools(w, dtype=kv_dtype)
    if poison_tail and w.decode_steps > 0:
        # rows the decode steps will append must come from ckv_append, not from the prefill image
        ps = w.page_size
        for s in range(w.batch):
            n0 = int(lens[s])
            for t in range(n0, n0 + w.decode_steps):
                pg = int(table[s, t // ps])
                k_pool[pg, :, t % ps] = float("nan")
                v_pool[pg, :, t % ps] = float("nan")
    dev = torch.device("cuda")
    max_blocks = synth.pages_per_seq(w) * w.page_size // w.block_size
    ckv = binding.CompKV(w.num_q_heads, w.num_kv_heads, max_batch=w.batch, max_blocks_per_seq=max_blocks,
                         num_pages=k_pool.shape[0], block_size=w.block_size,
                         var_groups=var_groups or w.var_groups, group_layout=group_layout,
                         kv_dtype=binding.CKV_BF16 if kv_dtype == torch.bfloat16 else binding.CKV_F32,
                         sink_blocks=sink, recent_blocks=recent, sm_scale=sm_scale, variant=variant,
                         stat_bf16=stat_bf16)
    return Device(w, ckv, k_pool.to(dev), v_pool.to(dev), table.to(dev), lens.to(dev),
                  int(lens.max()), kv_dtype)


def dev_q(d: Device, step: int = 0) -> torch.Tensor:
    return torch.from_numpy(synth.queries(d.w, step)).to(d.dtype).cuda()


def unit_inputs(w: synth.Workload, s: int, h: int, n: int, step: int = 0):
    """(q [G][d], K [n][d], V [n][d]) of one unit with the cache cut at n tokens."""
    k, v = synth.unit_kv(w, s, h)
    q = synth.queries(w, step)[s, h * w.group:(h + 1) * w.group]
    return np.ascontiguousarray(q), np.ascontiguousarray(k[:n]), np.ascontiguousarray(v[:n])


def rel_inf(a: np.ndarray, ref: np.ndarray) -> float:
    """max over rows of |a - ref|_inf / |ref|_inf."""
    a = np.asarray(a, np.float64).reshape(-1, a.shape[-1]); ref = np.asarray(ref, np.float64).reshape(a.shape)
    return float(np.max(np.abs(a - ref).max(1) / np.maximum(np.abs(ref).max(1), 1e-30)))


def check_stats(st: O.Stats, kmean, dbar, vmean, K: np.ndarray, V: np.ndarray) -> None:
    x = len(st.cnt)
    kscale = float(np.abs(K).max()); vscale = float(np.abs(V).max())
    km, db, vm = (t[:x].double().cpu().numpy() for t in (kmean, dbar, vmean))
    assert np.all(np.abs(km - st.kmean) <= STATS_RTOL * (np.abs(st.kmean) + kscale))
    assert np.all(np.abs(vm - st.vmean) <= STATS_RTOL * (np.abs(st.vmean) + vscale))
    # variances: relative to the block's own scale (largest group variance of the block), never below 1e-5 relative
    ref_scale = st.Dbar.max(axis=1, keepdims=True)
    assert np.all(np.abs(db - st.Dbar) <= STATS_RTOL * (np.abs(st.Dbar) + ref_scale) + 1e-12)


def round_stats_bf16(st: O.Stats) -> O.Stats:
    """The oracle's summaries with mean keys and mean values rounded to bf16 (variances untouched)."""
    import dataclasses
    km = synth.round_bf16_(np.ascontiguousarray(st.kmean, dtype=np.float32)).astype(np.float64)
    vm = synth.round_bf16_(np.ascontiguousarray(st.vmean, dtype=np.float32)).astype(np.float64)
    return dataclasses.replace(st, kmean=km, vmean=vm)


def check_scores(gpu_scores: np.ndarray, sc: O.Scores, rtol: float = SCORE_RTOL) -> None:
    ref = sc.S
    got = gpu_scores[:len(ref)]
    assert np.all(np.isfinite(got)) and np.all(got >= 0.0)
    if ref.max() == 0.0:            # no within-block variance anywhere: every score is exactly zero
        assert np.all(got == 0.0)
        return
    big = ref >= 1e-30 * ref.max()
    rel = np.abs(got[big] - ref[big]) / ref[big]
    assert rel.max() <= rtol, "score mismatch %.3g" % rel.max()


def check_ids(gpu_ids: Sequence[int], ref_ids: Sequence[int], S: np.ndarray, K: int, sink: int = 1,
              recent: int = 2, tie_rtol: float = TIE_RTOL) -> bool:
    """Selected ids must equal the oracle's, except on blocks whose oracle score is within TIE_RTOL
    (relative) of the threshold score.  Returns True when the sets are identical."""
    gpu_ids = [int(b) for b in gpu_ids]
    assert gpu_ids == sorted(set(gpu_ids)), "ids must be ascending and unique"
    assert len(gpu_ids) == len(ref_ids)
    if list(ref_ids) == gpu_ids:
        return True
    x = len(S)
    mand = {b for b in range(x) if b < sink or b >= x - recent}
    assert mand <= set(gpu_ids)
    ranked = sorted((S[b] for b in range(x) if b not in mand), reverse=True)
    tau = ranked[K - len(mand) - 1]
    for b in set(gpu_ids) ^ set(int(i) for i in ref_ids):
        assert abs(S[b] - tau) <= tie_rtol * tau, "block %d differs and is not a near tie (%.6g vs %.6g)" % (b, S[b], tau)
    return False


def check_unit_decode(d: Device, s: int, h: int, n: int, step: int, budget: int, out, lse, ids, cnt,
                      scores=None, var_groups: Optional[int] = None, group_layout: int = 1, sink: int = 1,
                      recent: int = 2, scale: Optional[float] = None, variant: int = 0,
                      stat_bf16: bool = False) -> Dict[str, float]:
    """Compare one unit of a finished ckv_decode with the oracle on the same inputs.

    variant: the ablation bits the context was created with (1: first-order mass, 2: rank by mass, 4: drop);
    the oracle is run with the matching switches."""
    w = d.w
    G = w.group
    q, K, V = unit_inputs(w, s, h, n, step)
    st = O.stats(K, V, w.block_size, var_groups or w.var_groups, group_layout)
    if stat_bf16:
        st = round_stats_bf16(st)
    sc = O.scores(q, st, scale, mass_order=1 if variant & 1 else 2, outer_var=0 if variant & 2 else 1)
    kblocks = budget // w.block_size
    ref_ids = O.select(sc.S, kblocks, sink, recent)
    nsel = int(cnt[s, h])
    gpu_ids = ids[s, h, :nsel].cpu().numpy()
    assert nsel == len(ref_ids)
    assert np.all(ids[s, h, nsel:].cpu().numpy() == -1)
    if scores is not None:
        check_scores(scores[s, h].double().cpu().numpy(), sc, SCORE_RTOL_STAT_BF16 if stat_bf16 else SCORE_RTOL)
    same = check_ids(gpu_ids, ref_ids, sc.S, kblocks, sink, recent, SCORE_RTOL_STAT_BF16 if stat_bf16 else TIE_RTOL)
    # when the sets differ only by near ties, the output is checked against the oracle on the GPU's ids
    ref_out, ref_lse = O.sparse(q, K, V, st, ref_ids if same else gpu_ids, scale, drop=bool(variant & 4))
    got = out[s, h * G:(h + 1) * G].double().cpu().numpy()
    err = rel_inf(got, ref_out)
    assert err <= OUT_TOL[d.dtype], "output error %.3g" % err
    got_lse = lse[s, h * G:(h + 1) * G].double().cpu().numpy()
    lerr = float(np.abs(got_lse - ref_lse).max())
    ltol = LSE_ATOL_STAT_BF16 if stat_bf16 else LSE_ATOL[d.dtype]
    assert lerr <= ltol * max(1.0, float(np.abs(ref_lse).max())), "lse error %.3g" % lerr
    return {"out_err": err, "lse_err": lerr, "ids_identical": float(same)}
