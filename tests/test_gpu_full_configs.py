"""GPU parity at the full sizes of the five benchmark configurations (the oracle computes one unit at a time, a
thread per unit), in the launch configuration the bench times (CUDA-graph replay of append + decode where the
configuration has decode steps).  The machinery that only exists at these sizes -- the scan's partial entries per
(CTA, unit), the tail CTAs' rounds, the cluster merge -- is per unit, so the 128K configuration checks EVERY unit at
its first and last step, the ragged one a unit of every sequence, the sweep every head at one budget per block
size; the steps and budgets in between check sampled units."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import compkv_oracle as O
from paper_2609_26300_b200 import synth
from paper_2609_26300_b200.runner import GraphStep

from helpers import OUT_TOL, check_stats, check_unit_decode, dev_q, rel_inf, setup, unit_inputs

pytestmark = pytest.mark.gpu


def check_units(units, fn):
    """fn(s, h) for every unit, a few at a time (the oracle is C called through ctypes: threads run in parallel)."""
    with ThreadPoolExecutor(min(8, os.cpu_count() or 1)) as ex:
        return list(ex.map(lambda u: fn(*u), units))


def test_config2_llama_32k():
    w = synth.CONFIGS[2]
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt = d.ckv.decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
    scores = d.ckv.copy_scores(w.batch)
    dout, dlse = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    assert cnt.cpu().tolist() == [[64] * 8]
    km, db, vm = d.ckv.export_stats()
    G = w.group
    for h in (0, 3, 7):
        check_unit_decode(d, 0, h, w.ctx, 0, w.budget_tokens, out, lse, ids, cnt, scores)
        q, K, V = unit_inputs(w, 0, h, w.ctx)
        check_stats(O.stats(K, V, 16), km[0, h], db[0, h], vm[0, h], K, V)
        ref, _ = O.dense(q, K, V)
        assert rel_inf(dout[0, h * G:(h + 1) * G].double().cpu().numpy(), ref) <= OUT_TOL[d.dtype]


def test_config3_llama_128k_batch4_64_decode_steps():
    w = synth.CONFIGS[3]
    d = setup(w)
    n0 = w.ctx
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, n0)
    step = GraphStep(d.ckv, d.k_pool, d.v_pool, d.table, d.lens, n0 + w.decode_steps, w.budget_tokens, w.batch)
    check_steps = {0, 1, 15, 16, 17, 31, 32, 63}
    sample = [(0, 0), (3, 5)]
    every = [(s, h) for s in range(w.batch) for h in range(w.num_kv_heads)]   # all 32 units at the first and last step
    for t in range(w.decode_steps):
        k_new, v_new = synth.appended_rows(w, t)
        step.set_inputs(torch.from_numpy(synth.queries(w, t)).bfloat16().cuda(),
                        torch.from_numpy(k_new).bfloat16().cuda(), torch.from_numpy(v_new).bfloat16().cuda())
        out, lse, ids, cnt = step.replay()
        if t in check_steps:
            scores = d.ckv.copy_scores(w.batch)
            torch.cuda.synchronize()
            assert cnt.cpu().tolist() == [[128] * 8] * 4
            res = check_units(every if t in (0, 63) else sample,
                              lambda s, h: check_unit_decode(d, s, h, n0 + t + 1, t, w.budget_tokens, out, lse, ids, cnt, scores))
            if t in (0, 63):
                print("config 3, step %d: ids identical to the oracle's on %d of %d units, worst output error %.2e"
                      % (t, sum(int(r["ids_identical"]) for r in res), len(res), max(r["out_err"] for r in res)))
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    assert d.lens.cpu().tolist() == [n0 + 64] * 4
    # summaries after 64 appends equal the oracle's over the longer cache
    km, db, vm = d.ckv.export_stats()
    for s, h in sample:
        _, K, V = unit_inputs(w, s, h, n0 + 64)
        check_stats(O.stats(K, V, 16), km[s, h], db[s, h], vm[s, h], K, V)


def test_config4_qwen_ragged_batch16_group8():
    w = synth.CONFIGS[4]
    d = setup(w)
    lens = d.lens.cpu().numpy()
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt = d.ckv.decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
    scores = d.ckv.copy_scores(w.batch)
    dout, _ = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    assert bool((cnt == 64).all())
    G = w.group
    # a unit of every sequence (the shortest and the longest among them), heads spread over the eight KV heads
    units = [(s, (3 * s + 1) % w.num_kv_heads) for s in range(w.batch)]
    assert int(lens.argmin()) in [s for s, _ in units] and int(lens.argmax()) in [s for s, _ in units]

    def one(s, h):
        r = check_unit_decode(d, s, h, int(lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores)
        q, K, V = unit_inputs(w, s, h, int(lens[s]))
        ref, _ = O.dense(q, K, V)
        assert rel_inf(dout[s, h * G:(h + 1) * G].double().cpu().numpy(), ref) <= OUT_TOL[d.dtype]
        return r
    res = check_units(units, one)
    print("config 4: ids identical to the oracle's on %d of %d units" % (sum(int(r["ids_identical"]) for r in res), len(res)))


@pytest.mark.parametrize("bs", synth.SWEEP_BLOCK_SIZES)
def test_config5_sweep_128k(bs):
    w = synth.CONFIGS[5].with_(block_size=bs)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    h = 2
    q, K, V = unit_inputs(w, 0, h, w.ctx)
    km, db, vm = d.ckv.export_stats()
    check_stats(O.stats(K, V, bs), km[0, h], db[0, h], vm[0, h], K, V)
    for budget in synth.SWEEP_BUDGETS:
        out, lse, ids, cnt = d.ckv.decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len, budget)
        scores = d.ckv.copy_scores(w.batch)
        torch.cuda.synchronize()
        assert cnt.cpu().tolist() == [[budget // bs] * 8]
        heads = range(w.num_kv_heads) if budget == 2048 else [h]   # every head at one budget per block size
        check_units([(0, hh) for hh in heads],
                    lambda s, hh: check_unit_decode(d, s, hh, w.ctx, 0, budget, out, lse, ids, cnt, scores))
    assert d.ckv.read_status() == 0


@pytest.mark.parametrize("kw,ck", [(dict(var_groups=128), dict(var_groups=128)),
                                   (dict(stat_bf16=1), dict(stat_bf16=True))])
def test_config2_other_layouts(kw, ck):
    """The 32K configuration at the r = d operating point and with bf16 summaries, a few decode steps each."""
    w = synth.CONFIGS[2].with_(decode_steps=3)
    d = setup(w, **kw)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    for t in range(3):
        k_new, v_new = synth.appended_rows(w, t)
        out, lse, ids, cnt = d.ckv.step(torch.from_numpy(synth.queries(w, t)).bfloat16().cuda(),
                                        torch.from_numpy(k_new).bfloat16().cuda(), torch.from_numpy(v_new).bfloat16().cuda(),
                                        d.k_pool, d.v_pool, d.table, d.lens, w.ctx + t + 1, w.budget_tokens)
        scores = d.ckv.copy_scores(w.batch)
        torch.cuda.synchronize()
        assert d.ckv.read_status() == 0
        for h in (1, 6):
            check_unit_decode(d, 0, h, w.ctx + t + 1, t, w.budget_tokens, out, lse, ids, cnt, scores, **ck)


@pytest.mark.parametrize("cfg", [2, 3])
def test_results_are_a_pure_function_of_the_inputs(cfg):
    """The same decode twice, and the same dense decode twice, on a full-size cache (148 scan CTAs, clusters of
    eight splits, counter-based merges): every output bit, id and score repeats."""
    w = synth.CONFIGS[cfg]
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    q = dev_q(d)
    runs = []
    for _ in range(3):
        out, lse, ids, cnt = d.ckv.decode(q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
        scores = d.ckv.copy_scores(w.batch)
        dout, dlse = d.ckv.dense_decode(q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
        torch.cuda.synchronize()
        runs.append([t.clone() for t in (out, lse, ids, cnt, scores, dout, dlse)])
    for r in runs[1:]:
        for x, y in zip(runs[0], r):
            assert torch.equal(x, y)
    assert d.ckv.read_status() == 0


def test_config4_qwen_steps_in_tail_mode():
    """The ragged 16-sequence, group-of-8 configuration stepped with ckv_step: at this size the library runs the
    append inside the scan launch (16 tail CTAs, 128 units), clusters of two attention splits per unit."""
    w = synth.CONFIGS[4].with_(decode_steps=6)
    d = setup(w)
    lens0 = d.lens.cpu().numpy().copy()
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    sample = [(int(lens0.argmin()), 1), (int(lens0.argmax()), 6), (7, 3)]
    for t in range(6):
        k_new, v_new = synth.appended_rows(w, t)
        n_before = d.ckv.launch_count()
        out, lse, ids, cnt = d.ckv.step(torch.from_numpy(synth.queries(w, t)).bfloat16().cuda(),
                                        torch.from_numpy(k_new).bfloat16().cuda(),
                                        torch.from_numpy(v_new).bfloat16().cuda(), d.k_pool, d.v_pool, d.table,
                                        d.lens, d.max_len + t + 1, w.budget_tokens)
        assert d.ckv.launch_count() - n_before == 3
        if t in (0, 5):
            scores = d.ckv.copy_scores(w.batch)
            torch.cuda.synchronize()
            for s, h in sample:
                check_unit_decode(d, s, h, int(lens0[s]) + t + 1, t, w.budget_tokens, out, lse, ids, cnt, scores)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    assert np.array_equal(d.lens.cpu().numpy(), lens0 + 6)
