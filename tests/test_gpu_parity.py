"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Small cases compare every unit element by element; the full-size configurations compare
sampled units (the oracle computes a unit in well under a second)."""
import numpy as np
import pytest
import torch

from oracle import compkv_oracle as O
import helpers
from paper_2609_26300_b200 import synth

from helpers import (OUT_TOL, check_ids, check_stats, check_unit_decode, dev_q, rel_inf, setup, unit_inputs)

pytestmark = pytest.mark.gpu

TOY = synth.CONFIGS[1]


def small(**kw):
    base = dict(batch=2, num_q_heads=8, num_kv_heads=2, ctx=16 * 70 + 5, budget_tokens=16 * 12, needles=4,
                outlier_dims=2, decode_steps=3, name="small")
    base.update(kw)
    return TOY.with_(**base)


def all_units(w):
    return [(s, h) for s in range(w.batch) for h in range(w.num_kv_heads)]


def run_decode(d, budget, step=0, max_len=None):
    q = dev_q(d, step)
    out, lse, ids, cnt = d.ckv.decode(q, d.k_pool, d.v_pool, d.table, d.lens, max_len or d.max_len, budget)
    scores = d.ckv.copy_scores(d.w.batch)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    return out, lse, ids, cnt, scores


# ---- stats --------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("bs", [16, 32, 64])
@pytest.mark.parametrize("r,layout", [(4, 1), (4, 0), (128, 1), (1, 1), (32, 0)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_stats_build(bs, r, layout, dtype):
    w = small(block_size=bs, ctx_min=16 * 20 + 1, ctx=16 * 70 + 5)   # ragged lengths, partial last blocks
    d = setup(w, dtype, var_groups=r, group_layout=layout)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    km, db, vm = d.ckv.export_stats()
    lens = d.lens.cpu().numpy()
    for s, h in all_units(w):
        _, K, V = unit_inputs(w, s, h, int(lens[s]))
        st = O.stats(K, V, bs, r, layout)
        check_stats(st, km[s, h], db[s, h], vm[s, h], K, V)
    assert d.ckv.read_status() == 0


@pytest.mark.parametrize("bs", [32, 64])
def test_blocks_of_several_pages_join_their_pages_exactly(bs):
    """Closed form for the pairwise joining of a block's pages (Eq. 8 over a block longer than a page): every
    16-token page holds one repeated key row, page p of a block at level p + 1 in every coordinate.  The block mean
    is then the mean of the levels and the variance their population variance -- ((n^2 - 1) / 12 for levels 1..n, all
    of it the joining term, since no page has any variance of its own) -- both exactly representable."""
    w = small(batch=1, num_q_heads=4, num_kv_heads=1, block_size=bs, ctx=bs * 6, decode_steps=0, needles=0,
              outlier_dims=0, shuffle_pages=False)
    d = setup(w, var_groups=4)
    ppb = bs // 16
    for page in range(d.k_pool.shape[0]):
        d.k_pool[page] = float(page % ppb + 1)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    km, db, vm = d.ckv.export_stats()
    mean = (ppb + 1) / 2.0
    var = (ppb * ppb - 1) / 12.0
    assert torch.equal(km[0, 0, :6].cpu(), torch.full((6, 128), mean))
    assert torch.equal(db[0, 0, :6].cpu(), torch.full((6, 4), var))
    assert d.ckv.read_status() == 0


@pytest.mark.parametrize("bs", [16, 32])
def test_append_equals_rebuild_bit_for_bit(bs):
    steps = 40   # crosses block boundaries: a filled block, a rollover, a one-token block
    w = small(block_size=bs, ctx=16 * 9 + 13, decode_steps=steps)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    n0 = int(d.lens[0])
    for t in range(steps):
        k_new, v_new = synth.appended_rows(w, t)
        d.ckv.append(d.k_pool, d.v_pool, d.table, d.lens,
                     torch.from_numpy(k_new).to(d.dtype).cuda(), torch.from_numpy(v_new).to(d.dtype).cuda())
    torch.cuda.synchronize()
    assert d.lens.cpu().tolist() == [n0 + steps] * w.batch
    km, db, vm = (t.clone() for t in d.ckv.export_stats())
    # the appended rows are now in the cache: a fresh build over the longer cache must agree exactly
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, n0 + steps)
    torch.cuda.synchronize()
    km2, db2, vm2 = d.ckv.export_stats()
    x = -(-(n0 + steps) // bs)
    assert torch.equal(km[:, :, :x], km2[:, :, :x]) and torch.equal(db[:, :, :x], db2[:, :, :x])
    assert torch.equal(vm[:, :, :x], vm2[:, :, :x])
    for s, h in all_units(w):
        _, K, V = unit_inputs(w, s, h, n0 + steps)
        check_stats(O.stats(K, V, bs), km[s, h], db[s, h], vm[s, h], K, V)
    assert d.ckv.read_status() == 0


# ---- decode: small cases, every unit ------------------------------------------------------------------------------

@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (8, 2), (16, 2)])   # G = 1, 2, 4, 8
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_decode_small_all_group_sizes(hq, hkv, dtype):
    w = small(num_q_heads=hq, num_kv_heads=hkv, ctx_min=16 * 30, ctx=16 * 70 + 5)
    d = setup(w, dtype)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    lens = d.lens.cpu().numpy()
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores)


@pytest.mark.parametrize("bs,budget", [(32, 32 * 6), (64, 64 * 4), (16, 16 * 3), (16, 16 * 37)])
@pytest.mark.parametrize("r,layout", [(4, 1), (128, 1), (8, 0)])
def test_decode_small_block_sizes_and_groups(bs, budget, r, layout):
    w = small(block_size=bs, budget_tokens=budget, ctx=16 * 90 + 7)
    d = setup(w, var_groups=r, group_layout=layout)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, budget)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, budget, out, lse, ids, cnt, scores, var_groups=r,
                          group_layout=layout)


@pytest.mark.parametrize("variant", [1, 2, 4, 3, 7])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_decode_scorer_and_merge_ablations(variant, dtype):
    """The ablations of Sec. 5.3 / App. A.6 as layout flags: first-order mass, ranking by mass alone, Drop."""
    w = small(block_size=16, budget_tokens=16 * 12, ctx=16 * 70 + 5)
    d = setup(w, dtype, variant=variant)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores, variant=variant)


@pytest.mark.parametrize("bs,hq", [(16, 8), (32, 8), (64, 8), (16, 16), (16, 2)])
def test_bf16_summaries_layout(bs, hq):
    """ckv_layout.stat_bf16: mean keys / mean values stored as bf16 (half the summary bytes).  The oracle runs on
    its own summaries rounded to bf16; stats must match to a bf16 ulp, the step within the layout's tolerances."""
    w = small(block_size=bs, budget_tokens=bs * 9, ctx=16 * 90 + 7, num_q_heads=hq, decode_steps=20)
    d = setup(w, stat_bf16=1)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    km, db, vm = d.ckv.export_stats(w.batch)
    for s, h in all_units(w):
        n = int(d.lens[s])
        _, K, V = unit_inputs(w, s, h, n)
        st = helpers.round_stats_bf16(O.stats(K, V, bs))
        x = len(st.cnt)
        for got, ref in ((km[s, h, :x], st.kmean), (vm[s, h, :x], st.vmean)):
            err = np.abs(got.double().cpu().numpy() - ref)
            assert np.all(err <= 2.0 ** -7 * np.abs(ref) + 1e-30)          # at most one bf16 ulp (a rounding flip)
            assert np.mean(err == 0.0) > 0.99                                # and almost always none
        assert np.allclose(db[s, h, :x].double().cpu().numpy(), st.Dbar, rtol=1e-5, atol=1e-12)
    checked, identical = decode_loop(d, 20, w.budget_tokens, set(range(20)), all_units(w), fused=True, stat_bf16=True)
    # this layout's near-tie rule is 500 times wider than the default one (helpers.SCORE_RTOL_STAT_BF16): say how
    # often it was needed at all (run with -s to see it), and require that it is the exception
    print("bf16 summaries, block %d, %d heads: selected ids identical to the oracle's on %d of %d unit-steps"
          % (bs, hq, identical, checked))
    assert identical >= 0.9 * checked


@pytest.mark.parametrize("blocks", [70, 71, 72, 73])
def test_decode_with_odd_and_even_row_strides(blocks):
    """max_blocks_per_seq = 70 .. 73: the per-block outputs of the scan are stored in pairs only when their rows start
    on 8-byte boundaries; both forms must give the same step."""
    w = small(ctx=16 * blocks - 3, decode_steps=0)
    d = setup(w)
    assert d.ckv.layout.max_blocks_per_seq == blocks
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores)


def test_decode_toy_config_fp32_and_bf16():
    for dtype in (torch.float32, torch.bfloat16):
        d = setup(TOY, dtype)
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
        out, lse, ids, cnt, scores = run_decode(d, TOY.budget_tokens)
        res = check_unit_decode(d, 0, 0, TOY.ctx, 0, TOY.budget_tokens, out, lse, ids, cnt, scores)
        assert int(cnt[0, 0]) == 16


def test_custom_scale_and_mandatory_counts():
    w = small()
    d = setup(w, sink=2, recent=3, sm_scale=0.05)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores, sink=2, recent=3,
                          scale=0.05)
        got = ids[s, h, :int(cnt[s, h])].tolist()
        x = -(-int(d.lens[s]) // 16)
        assert got[:2] == [0, 1] and got[-3:] == [x - 3, x - 2, x - 1]


# ---- special cases the method fixes -------------------------------------------------------------------------------------

def test_select_all_equals_dense_kernel_and_oracle():
    w = small(ctx=16 * 20 + 3, budget_tokens=16 * 32)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, _ = run_decode(d, w.budget_tokens)
    dout, dlse = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    x = 21
    assert cnt.cpu().tolist() == [[x] * w.num_kv_heads] * w.batch
    assert ids[0, 0, :x].tolist() == list(range(x)) and ids[0, 0, x:].tolist() == [-1] * (32 - x)
    for s, h in all_units(w):
        q, K, V = unit_inputs(w, s, h, int(d.lens[s]))
        ref, ref_lse = O.dense(q, K, V)
        G = w.group
        for o, l in ((out, lse), (dout, dlse)):
            assert rel_inf(o[s, h * G:(h + 1) * G].double().cpu().numpy(), ref) <= OUT_TOL[d.dtype]
            assert np.abs(l[s, h * G:(h + 1) * G].double().cpu().numpy() - ref_lse).max() <= 1e-4


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_dense_decode_parity(dtype):
    w = small(ctx_min=16 * 10, ctx=16 * 300 + 9, batch=3)
    d = setup(w, dtype)
    out, lse = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    G = w.group
    for s, h in all_units(w):
        q, K, V = unit_inputs(w, s, h, int(d.lens[s]))
        ref, ref_lse = O.dense(q, K, V)
        assert rel_inf(out[s, h * G:(h + 1) * G].double().cpu().numpy(), ref) <= OUT_TOL[dtype]
        assert np.abs(lse[s, h * G:(h + 1) * G].double().cpu().numpy() - ref_lse).max() <= 1e-4
    assert d.ckv.read_status() == 0


def test_constant_key_blocks_make_any_selection_exact():
    """Identical keys inside every block: mean compensation is exact, so the sparse output equals dense
    attention whatever is selected (fp32 layout, tight tolerance)."""
    w = small(batch=1, num_q_heads=4, num_kv_heads=1, ctx=16 * 40, decode_steps=0, needles=0, outlier_dims=0)
    d = setup(w, torch.float32)
    first = d.k_pool[:, :, :1, :].clone()
    d.k_pool.copy_(first.expand_as(d.k_pool))
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, 16 * 5)
    dout, dlse = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert int(cnt[0, 0]) == 5
    assert float(scores[0, 0, :40].abs().max()) < 1e-9      # no within-block variance => zero scores
    assert ids[0, 0, :5].tolist() == [0, 1, 2, 38, 39]       # all tied: lowest ids after the mandatory ones
    assert rel_inf(out[0].double().cpu().numpy(), dout[0].double().cpu().numpy()) <= 1e-5
    assert float((lse - dlse).abs().max()) <= 1e-5


def test_exact_ties_go_to_lower_block_ids():
    """Blocks with identical contents score identically on the GPU and in the oracle: stable order decides."""
    w = small(batch=1, num_q_heads=4, num_kv_heads=1, ctx=16 * 64, decode_steps=0, needles=0, outlier_dims=0,
              shuffle_pages=False)
    d = setup(w)
    # make blocks 8..39 copies of blocks 40..71 -> pairs of exactly tied scores (page == block, unshuffled)
    d.k_pool[8:36] = d.k_pool[36:64]
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, 16 * 20)
    sc = scores[0, 0, :64].cpu().numpy()
    assert np.array_equal(sc[8:35], sc[36:63])
    # the last block of a sequence is scored by the launch's tail CTAs (plain FMAs, not tensor-core tiles): its
    # pair agrees to rounding, not bit for bit; it is a mandatory block, so no tie is decided by it
    assert abs(sc[35] - sc[63]) <= 1e-6 * abs(sc[63])
    K = d.k_pool[:64, 0].float().reshape(-1, 128).cpu().numpy()
    V = d.v_pool[:64, 0].float().reshape(-1, 128).cpu().numpy()
    q = synth.queries(w)[0]
    st = O.stats(K, V, 16)
    osc = O.scores(q, st)
    assert np.array_equal(osc.S[8:36], osc.S[36:64])
    ref_ids = O.select(osc.S, 20)
    got = ids[0, 0, :int(cnt[0, 0])].cpu().numpy()
    check_ids(got, ref_ids, osc.S, 20)
    # among an exactly tied pair the lower id must be the one taken (or both)
    for b in range(8, 34):          # 62 and 63 (= 34 + 28, 35 + 28) are mandatory, so start the pairs below them
        if (b + 28) in got:
            assert b in got


def test_mean_values_read_as_hi_halves_worst_case():
    """The decode step of the default layout reads the mean values at bf16 precision (their hi halves).  Worst case
    for that: every block mean sits half a bf16 step above a representable value, in every coordinate and with the
    same sign (tokens alternate between 1 and 1 + 2^-7, mean 1 + 2^-8), and a small budget leaves most of the mass
    to the compensation term.  The output may then be off by that half step, 2^-8 relative, on top of the half step
    of its own bf16 rounding -- no more."""
    w = small(batch=1, num_q_heads=4, num_kv_heads=1, ctx=16 * 96, decode_steps=0, needles=0, outlier_dims=0,
              shuffle_pages=False)
    d = setup(w)
    d.v_pool[:, :, 0::2, :] = 1.0
    d.v_pool[:, :, 1::2, :] = 1.0 + 2.0 ** -7
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    km, db, vm = d.ckv.export_stats()
    assert torch.equal(vm[0, 0, :96].cpu(), torch.full((96, 128), 1.0 + 2.0 ** -8))   # the stored summaries keep it
    out, lse, ids, cnt, scores = run_decode(d, 16 * 6)
    K = d.k_pool[:96, 0].float().reshape(-1, 128).cpu().numpy()
    V = d.v_pool[:96, 0].float().reshape(-1, 128).cpu().numpy()
    q = synth.queries(w)[0]
    st = O.stats(K, V, 16)
    osc = O.scores(q, st)
    ref_ids = O.select(osc.S, 6)
    got = ids[0, 0, :int(cnt[0, 0])].cpu().numpy()
    same = check_ids(got, ref_ids, osc.S, 6)
    ref_out, ref_lse = O.sparse(q, K, V, st, ref_ids if same else got)
    err = rel_inf(out[0].double().cpu().numpy(), ref_out)
    assert err <= 2.0 ** -8 + 2.0 ** -8 + 1e-4, err
    assert float(np.abs(lse[0].double().cpu().numpy() - ref_lse).max()) <= 1e-4


# ---- edge cases ---------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 15, 16, 17, 47, 48, 49])
def test_tiny_sequences(n):
    w = small(batch=1, ctx=n, decode_steps=0, needles=0, budget_tokens=16 * 3)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, 16 * 3)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, n, 0, 16 * 3, out, lse, ids, cnt, scores)
    dout, _ = d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    G = w.group
    q, K, V = unit_inputs(w, 0, 1, n)
    assert rel_inf(dout[0, G:2 * G].double().cpu().numpy(), O.dense(q, K, V)[0]) <= OUT_TOL[d.dtype]


def test_empty_sequence_in_batch():
    w = small(batch=2, decode_steps=0)
    d = setup(w)
    d.lens[1] = 0
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    assert cnt[1].tolist() == [0] * w.num_kv_heads and bool((ids[1] == -1).all())
    assert float(out[1].float().abs().max()) == 0.0
    for h in range(w.num_kv_heads):
        check_unit_decode(d, 0, h, int(d.lens[0]), 0, w.budget_tokens, out, lse, ids, cnt, scores)


def test_budget_errors_and_argument_checks():
    from paper_2609_26300_b200 import binding
    w = small(decode_steps=0)
    d = setup(w)
    q = dev_q(d)
    with pytest.raises(binding.CompKVError) as e:
        d.ckv.decode(q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len, 16 * 2)    # K = 2 < 3 mandatory blocks
    assert e.value.status == binding.CKV_ERR_BUDGET_TOO_SMALL
    with pytest.raises(binding.CompKVError) as e:
        d.ckv.decode(q, d.k_pool, d.v_pool, d.table, d.lens, 10 ** 8, 16 * 8)      # longer than the layout allows
    assert e.value.status == binding.CKV_ERR_INVALID_ARG
    with pytest.raises(binding.CompKVError):
        binding.CompKV(12, 4, 1, 8, 8)                                              # G = 3 unsupported
    with pytest.raises(binding.CompKVError):
        binding.CompKV(8, 2, 1, 8, 8, block_size=48)


def test_bad_page_id_sets_status_and_does_not_fault():
    w = small(batch=1, decode_steps=0)
    d = setup(w)
    from paper_2609_26300_b200 import binding
    d.table[0, 5] = d.k_pool.shape[0] + 7      # outside the pool: must be skipped, not dereferenced
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() & binding.CKV_DEV_BAD_PAGE
    d.ckv.dense_decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() & binding.CKV_DEV_BAD_PAGE
    assert d.ckv.read_status() == 0            # reading clears it


def test_bounded_wait_runs_out_and_the_context_recovers():
    """Failure detection without a fault: the scan's producer announces one shared-memory fill and never issues it
    (a test hook), the poll limit of the bounded waits is lowered to 2^10, and the step must RETURN with
    CKV_DEV_TIMEOUT in the status word -- nothing traps, nothing waits for ever, no copy is left in flight.  With the
    hook cleared, the next step on the same context is correct against the oracle."""
    from paper_2609_26300_b200 import binding
    w = small(batch=1, num_q_heads=4, num_kv_heads=1, ctx=16 * 60 + 3, budget_tokens=16 * 8, decode_steps=0)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    d.ckv.debug_set(1 << 10, binding.CKV_DEBUG_SKIP_FILL)
    d.ckv.decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
    torch.cuda.synchronize()                       # the launch came back
    st = d.ckv.read_status()
    assert st & binding.CKV_DEV_TIMEOUT, st
    assert d.ckv.read_status() == 0                # reading cleared it
    d.ckv.debug_set(0, 0)                          # default poll limit, no hook
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores)
    # the same through the fused step (the scan launch with its tail CTAs)
    d.ckv.set_tail_mode(binding.CKV_TAIL_ON)
    d.ckv.debug_set(1 << 10, binding.CKV_DEBUG_SKIP_FILL)
    d.ckv.decode(dev_q(d), d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
    torch.cuda.synchronize()
    assert d.ckv.read_status() & binding.CKV_DEV_TIMEOUT
    d.ckv.debug_set(0, 0)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    for s, h in all_units(w):
        check_unit_decode(d, s, h, int(d.lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores)


def test_append_past_capacity_sets_status():
    from paper_2609_26300_b200 import binding
    w = small(batch=1, ctx=16 * 4, decode_steps=0)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    z = torch.zeros(1, w.num_kv_heads, 128, dtype=d.dtype, device="cuda")
    d.ckv.append(d.k_pool, d.v_pool, d.table, d.lens, z, z)       # table has room for exactly ctx tokens
    torch.cuda.synchronize()
    assert d.ckv.read_status() & binding.CKV_DEV_SEQ_FULL
    assert int(d.lens[0]) == 16 * 4


# ---- decode steps with appends ----------------------------------------------------------------------------------------

def decode_loop(d, steps, budget, check_steps, sample_units, use_host_call=False, fused=False, tail_on=None, **ck):
    from paper_2609_26300_b200 import binding
    w = d.w
    # these caches are small: left to itself the library would take the two-call route for every step, so the
    # ckv_step tests switch tail mode (the append inside the scan launch) on explicitly
    if fused or tail_on:
        d.ckv.set_tail_mode(binding.CKV_TAIL_ON)
    n0 = d.lens.cpu().numpy().copy()
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    checked = identical = 0
    for t in range(steps):
        k_new, v_new = synth.appended_rows(w, t)
        q = synth.queries(w, t)
        max_len = d.max_len + t + 1
        if use_host_call:
            kcap = budget // w.block_size
            hq = torch.from_numpy(q).to(d.dtype).pin_memory()
            hk = torch.from_numpy(k_new).to(d.dtype).pin_memory(); hv = torch.from_numpy(v_new).to(d.dtype).pin_memory()
            ho = torch.empty(w.batch, w.num_q_heads, 128, dtype=d.dtype).pin_memory()
            hi = torch.empty(w.batch, w.num_kv_heads, kcap, dtype=torch.int32).pin_memory()
            hc = torch.empty(w.batch, w.num_kv_heads, dtype=torch.int32).pin_memory()
            d.ckv.step_host(hq, hk, hv, d.k_pool, d.v_pool, d.table, d.lens, max_len, budget, ho, hi, hc)
            out, ids, cnt = ho, hi, hc
            lse = None
        elif fused:   # ckv_step: the same step in one call
            out, lse, ids, cnt = d.ckv.step(torch.from_numpy(q).to(d.dtype).cuda(),
                                            torch.from_numpy(k_new).to(d.dtype).cuda(),
                                            torch.from_numpy(v_new).to(d.dtype).cuda(), d.k_pool, d.v_pool, d.table,
                                            d.lens, max_len, budget)
        else:
            d.ckv.append(d.k_pool, d.v_pool, d.table, d.lens, torch.from_numpy(k_new).to(d.dtype).cuda(),
                         torch.from_numpy(v_new).to(d.dtype).cuda())
            out, lse, ids, cnt = d.ckv.decode(torch.from_numpy(q).to(d.dtype).cuda(), d.k_pool, d.v_pool, d.table,
                                              d.lens, max_len, budget)
        if t in check_steps:
            scores = d.ckv.copy_scores(w.batch)
            torch.cuda.synchronize()
            for s, h in sample_units:
                if lse is None:   # the host call returns no lse: compare outputs and ids only
                    G = w.group
                    qq, K, V = unit_inputs(w, s, h, int(n0[s]) + t + 1, t)
                    st = O.stats(K, V, w.block_size)
                    sc = O.scores(qq, st)
                    ref_ids = O.select(sc.S, budget // w.block_size)
                    got = ids[s, h, :int(cnt[s, h])].numpy()
                    same = check_ids(got, ref_ids, sc.S, budget // w.block_size)
                    ref, _ = O.sparse(qq, K, V, st, ref_ids if same else got)
                    assert rel_inf(out[s, h * G:(h + 1) * G].double().numpy(), ref) <= OUT_TOL[d.dtype]
                else:
                    res = check_unit_decode(d, s, h, int(n0[s]) + t + 1, t, budget, out, lse, ids, cnt, scores, **ck)
                    checked += 1
                    identical += int(res["ids_identical"])
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    assert np.array_equal(d.lens.cpu().numpy(), n0 + steps)
    return checked, identical


def test_decode_loop_small_with_appends():
    w = small(ctx_min=16 * 30 + 1, ctx=16 * 60, decode_steps=36)
    d = setup(w)
    decode_loop(d, 36, w.budget_tokens, set(range(36)), all_units(w))


@pytest.mark.parametrize("tail_on", [False, True])
@pytest.mark.parametrize("hq,stat_bf16", [(32, 0), (64, 0), (32, 1)])
def test_scan_ctas_that_span_many_units(hq, stat_bf16, tail_on):
    """Many short sequences: 320 units of two to three scan tiles each, so that a scan CTA's range spans three to
    six units -- more than it stages query rows for -- and its warps change units every few parts.  Every unit of
    a sample of sequences against the oracle, in both step arrangements."""
    from paper_2609_26300_b200 import binding
    w = small(batch=40, num_q_heads=hq, num_kv_heads=8, ctx_min=16 * 40 + 1, ctx=16 * 90 + 5, budget_tokens=16 * 10,
              decode_steps=0, needles=1)
    d = setup(w, stat_bf16=stat_bf16)
    d.ckv.set_tail_mode(binding.CKV_TAIL_ON if tail_on else binding.CKV_TAIL_OFF)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    out, lse, ids, cnt, scores = run_decode(d, w.budget_tokens)
    lens = d.lens.cpu().numpy()
    for s in (0, 7, 19, 33, 39):
        for h in range(w.num_kv_heads):
            check_unit_decode(d, s, h, int(lens[s]), 0, w.budget_tokens, out, lse, ids, cnt, scores,
                              stat_bf16=bool(stat_bf16))


def test_decode_loop_two_calls_in_tail_mode():
    """ckv_append + ckv_decode with the last block of every sequence left to the scan launch's tail CTAs."""
    w = small(ctx_min=16 * 30 + 1, ctx=16 * 60, decode_steps=20)
    d = setup(w)
    decode_loop(d, 20, w.budget_tokens, set(range(20)), all_units(w), tail_on=True)


@pytest.mark.parametrize("bs,r", [(16, 4), (32, 4), (64, 4), (16, 128), (16, 8), (16, 64), (16, 1), (32, 32)])
def test_fused_step_loop(bs, r):
    """ckv_step over block roll-overs, one-token blocks and ragged lengths: every unit, every step."""
    w = small(ctx_min=16 * 30 + 1, ctx=16 * 60, decode_steps=36, block_size=bs, budget_tokens=bs * 7)
    d = setup(w, var_groups=r)
    decode_loop(d, 36, w.budget_tokens, set(range(36)), all_units(w), fused=True, var_groups=r)


def test_fused_step_custom_scale_group_layout_and_mandatory_counts():
    """Tail mode with a logit scale of the caller's, contiguous coordinate groups, two sink and three recent blocks:
    the last block's terms come from the tail warps' own arithmetic and must follow the same layout switches."""
    w = small(ctx_min=16 * 25 + 3, ctx=16 * 50 + 9, decode_steps=18)
    d = setup(w, sink=2, recent=3, sm_scale=0.05, group_layout=0, var_groups=8)
    decode_loop(d, 18, w.budget_tokens, set(range(18)), all_units(w), fused=True, sink=2, recent=3, scale=0.05,
                group_layout=0, var_groups=8)


@pytest.mark.parametrize("hq,hkv", [(2, 2), (16, 2)])   # G = 1 and 8
def test_fused_step_group_sizes(hq, hkv):
    w = small(ctx=16 * 40 + 9, decode_steps=20, num_q_heads=hq, num_kv_heads=hkv)
    d = setup(w)
    decode_loop(d, 20, w.budget_tokens, set(range(20)), all_units(w), fused=True)


@pytest.mark.parametrize("variant", [1, 2, 4])
def test_fused_step_ablations(variant):
    w = small(ctx=16 * 40 + 15, decode_steps=6)
    d = setup(w, variant=variant)
    decode_loop(d, 6, w.budget_tokens, set(range(6)), all_units(w), fused=True, variant=variant)


def test_fused_step_from_short_and_single_block_sequences():
    """Sequences that start with one token / exactly one block: the scan has nothing or one block to cover."""
    for n in (1, 15, 16, 17):
        w = small(ctx=n, decode_steps=20, budget_tokens=16 * 4, needles=0)
        d = setup(w)
        decode_loop(d, 20, w.budget_tokens, set(range(20)), all_units(w), fused=True)


def test_fused_step_select_all_and_recent_zero_fallback():
    w = small(ctx=16 * 12 + 3, decode_steps=8, budget_tokens=16 * 64)     # K >= X: dense
    d = setup(w)
    decode_loop(d, 8, w.budget_tokens, set(range(8)), all_units(w), fused=True)
    w = small(ctx=16 * 40 + 3, decode_steps=8)
    d = setup(w, sink=1, recent=0)                                         # no mandatory tail block
    decode_loop(d, 8, w.budget_tokens, set(range(8)), all_units(w), fused=True, sink=1, recent=0)


def test_decode_loop_through_host_buffer_call():
    w = small(ctx=16 * 50 + 15, decode_steps=20)
    d = setup(w)
    decode_loop(d, 20, w.budget_tokens, {0, 1, 2, 16, 17, 19}, all_units(w), use_host_call=True)


def test_host_buffer_call_replayed_from_fixed_buffers():
    """A decode loop that reuses its pinned buffers on a stream of its own: ckv_step_host captures its second call
    and replays it afterwards (the length bound is rounded up inside); results equal ckv_step's, step by step."""
    w = small(ctx=16 * 40 + 3, decode_steps=24)
    a, b = setup(w), setup(w)
    kcap = w.budget_tokens // w.block_size
    for d in (a, b):
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    hq = torch.zeros(w.batch, w.num_q_heads, 128, dtype=a.dtype).pin_memory()
    hk = torch.zeros(w.batch, w.num_kv_heads, 128, dtype=a.dtype).pin_memory()
    hv = torch.zeros_like(hk).pin_memory()
    ho = torch.zeros_like(hq).pin_memory()
    hi = torch.zeros(w.batch, w.num_kv_heads, kcap, dtype=torch.int32).pin_memory()
    hc = torch.zeros(w.batch, w.num_kv_heads, dtype=torch.int32).pin_memory()
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    n_before = a.ckv.launch_count()
    for t in range(24):
        k_new, v_new = synth.appended_rows(w, t)
        q = synth.queries(w, t)
        hq.copy_(torch.from_numpy(q).to(a.dtype)); hk.copy_(torch.from_numpy(k_new).to(a.dtype))
        hv.copy_(torch.from_numpy(v_new).to(a.dtype))
        with torch.cuda.stream(side):
            a.ckv.step_host(hq, hk, hv, a.k_pool, a.v_pool, a.table, a.lens, a.max_len + t + 1, w.budget_tokens, ho, hi, hc)
        ob, lb, ib, cb = b.ckv.step(hq.cuda(), hk.cuda(), hv.cuda(), b.k_pool, b.v_pool, b.table, b.lens,
                                    b.max_len + t + 1, w.budget_tokens)
        torch.cuda.synchronize()
        assert torch.equal(ho, ob.cpu()) and torch.equal(hi, ib.cpu()) and torch.equal(hc, cb.cpu()), t
        assert torch.equal(a.lens, b.lens), t
    assert a.ckv.launch_count() - n_before == 24 * 6   # in, append, scan, select, attention, out: replays count too
    assert a.ckv.read_status() == 0 and b.ckv.read_status() == 0


def test_host_buffer_call_pinned_and_pageable_buffers_agree():
    """ckv_step_host moves pinned buffers with kernels of its own and pageable ones with copies: same results."""
    w = small(ctx=16 * 40 + 3, decode_steps=4, budget_tokens=16 * 9 + 16)   # 10 ids per unit: a 40-byte id row
    a, b = setup(w), setup(w)
    kcap = w.budget_tokens // w.block_size
    for d in (a, b):
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    for t in range(4):
        k_new, v_new = synth.appended_rows(w, t)
        q = synth.queries(w, t)
        res = []
        for d, pin in ((a, True), (b, False)):
            mk = (lambda x: x.pin_memory()) if pin else (lambda x: x)
            hq = mk(torch.from_numpy(q).to(d.dtype)); hk = mk(torch.from_numpy(k_new).to(d.dtype))
            hv = mk(torch.from_numpy(v_new).to(d.dtype))
            ho = mk(torch.zeros(w.batch, w.num_q_heads, 128, dtype=d.dtype))
            hi = mk(torch.zeros(w.batch, w.num_kv_heads, kcap, dtype=torch.int32))
            hc = mk(torch.zeros(w.batch, w.num_kv_heads, dtype=torch.int32))
            d.ckv.step_host(hq, hk, hv, d.k_pool, d.v_pool, d.table, d.lens, d.max_len + t + 1, w.budget_tokens,
                            ho, hi, hc)
            res.append((ho.clone(), hi.clone(), hc.clone()))
        for x, y in zip(*res):
            assert torch.equal(x, y), t
        assert int(res[0][2].min()) == kcap
    assert a.ckv.read_status() == 0 and b.ckv.read_status() == 0
