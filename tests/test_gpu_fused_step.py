"""The fused step (ckv_step: the new token's append rides in the scan launch) against the two-call sequence
ckv_append + ckv_decode on identical caches, and its corner cases: full sequences, more units than one round of
tail warps, fp32 pages, bf16 summaries."""
import pytest
import torch

from paper_2609_26300_b200 import binding, synth
from helpers import setup

pytestmark = pytest.mark.gpu

TOY = synth.CONFIGS[1]


def small(**kw):
    base = dict(batch=2, num_q_heads=8, num_kv_heads=2, ctx=16 * 70 + 5, budget_tokens=16 * 12, needles=4,
                outlier_dims=2, decode_steps=3, name="small")
    base.update(kw)
    return TOY.with_(**base)


def rows(d, t):
    k_new, v_new = synth.appended_rows(d.w, t)
    q = synth.queries(d.w, t)
    return (torch.from_numpy(q).to(d.dtype).cuda(), torch.from_numpy(k_new).to(d.dtype).cuda(),
            torch.from_numpy(v_new).to(d.dtype).cuda())


def run_both(w, steps, dtype=torch.bfloat16, step_launches=3, tail=binding.CKV_TAIL_ON, **layout):
    """Two identical caches: one stepped with ckv_step, one with ckv_append + ckv_decode.  The summaries, pages,
    lengths and selected ids must be identical; the outputs agree bit for bit (same kernels, same order).  The
    caches here are small, so the mode the library would pick by itself is the two-call one: tail mode (the
    append inside the scan launch) is switched on explicitly unless a test says otherwise."""
    a, b = setup(w, dtype, **layout), setup(w, dtype, **layout)
    for d in (a, b):
        d.ckv.set_tail_mode(tail)
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    for t in range(steps):
        q, kn, vn = rows(a, t)
        max_len = a.max_len + t + 1
        n_before = a.ckv.launch_count()
        oa, la, ia, ca = a.ckv.step(q, kn, vn, a.k_pool, a.v_pool, a.table, a.lens, max_len, w.budget_tokens)
        assert a.ckv.launch_count() - n_before == step_launches
        b.ckv.append(b.k_pool, b.v_pool, b.table, b.lens, kn, vn)
        ob, lb, ib, cb = b.ckv.decode(q, b.k_pool, b.v_pool, b.table, b.lens, max_len, w.budget_tokens)
        torch.cuda.synchronize()
        assert torch.equal(a.lens, b.lens), t
        assert torch.equal(ca, cb) and torch.equal(ia, ib), t
        assert torch.equal(oa, ob) and torch.equal(la, lb), t
        sa, sb = a.ckv.copy_scores(w.batch), b.ckv.copy_scores(w.batch)
        assert torch.equal(sa, sb), t
    torch.cuda.synchronize()
    assert torch.equal(a.k_pool, b.k_pool) and torch.equal(a.v_pool, b.v_pool)
    for x, y in zip(a.ckv.export_stats(), b.ckv.export_stats()):
        assert torch.equal(x, y)
    assert a.ckv.read_status() == 0 and b.ckv.read_status() == 0
    return a


@pytest.mark.parametrize("bs", [16, 32, 64])
def test_step_equals_append_then_decode(bs):
    w = small(block_size=bs, ctx_min=16 * 20 + 1, ctx=16 * 70 + 5, budget_tokens=bs * 7, decode_steps=40)
    run_both(w, 40)   # crosses block boundaries in every sequence: full block, roll-over, one-token block


@pytest.mark.parametrize("r,layout", [(128, 1), (8, 0), (1, 1)])
def test_step_equals_append_then_decode_variance_layouts(r, layout):
    w = small(ctx=16 * 33 + 14, decode_steps=20)
    run_both(w, 20, var_groups=r, group_layout=layout)


def test_step_equals_append_then_decode_fp32_pages():
    w = small(ctx=16 * 33 + 14, decode_steps=20)
    run_both(w, 20, dtype=torch.float32, step_launches=4)   # fp32 pages merge in a launch of their own


def test_step_equals_append_then_decode_bf16_summaries():
    w = small(ctx=16 * 33 + 14, decode_steps=20)
    run_both(w, 20, stat_bf16=1)


def test_step_launch_count_is_three():
    w = small(decode_steps=2)
    d = setup(w)
    d.ckv.set_tail_mode(binding.CKV_TAIL_ON)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    n0 = d.ckv.launch_count()
    q, kn, vn = rows(d, 0)
    d.ckv.step(q, kn, vn, d.k_pool, d.v_pool, d.table, d.lens, d.max_len + 1, w.budget_tokens)
    torch.cuda.synchronize()
    assert d.ckv.launch_count() - n0 == 3   # scan (with the append in its tail CTAs), select, attention + merge


def test_many_units_one_round_of_tail_warps():
    """72 units: nine tail CTAs, one unit per warp."""
    w = small(batch=9, num_q_heads=16, num_kv_heads=8, ctx_min=16 * 8 + 1, ctx=16 * 20 + 3, decode_steps=18,
              budget_tokens=16 * 6, needles=1)
    run_both(w, 18)


def test_more_units_than_one_round_of_tail_warps():
    """136 units: the tail warps go round twice."""
    w = small(batch=17, num_q_heads=8, num_kv_heads=8, ctx_min=16 * 8 + 1, ctx=16 * 20 + 3, decode_steps=6,
              budget_tokens=16 * 6, needles=0)
    run_both(w, 6)


def test_small_steps_take_the_two_call_route_by_default_and_agree_with_tail_mode():
    """Left to itself the library appends in a launch of its own when the scan is too short to hide the tail CTAs
    (four launches); the result agrees with tail mode to rounding: same ids, outputs within the bf16 tolerance."""
    w = small(ctx_min=16 * 20 + 1, ctx=16 * 70 + 5, decode_steps=10)
    a = run_both(w, 10, step_launches=4, tail=binding.CKV_TAIL_AUTO)
    b = run_both(w, 10, step_launches=3, tail=binding.CKV_TAIL_ON)
    q = torch.from_numpy(synth.queries(w, 9)).to(a.dtype).cuda()
    oa, la, ia, ca = a.ckv.decode(q, a.k_pool, a.v_pool, a.table, a.lens, a.max_len + 10, w.budget_tokens)
    ob, lb, ib, cb = b.ckv.decode(q, b.k_pool, b.v_pool, b.table, b.lens, b.max_len + 10, w.budget_tokens)
    torch.cuda.synchronize()
    assert torch.equal(ia, ib) and torch.equal(ca, cb)
    assert float((oa.float() - ob.float()).abs().max()) <= 2e-2 * float(ob.float().abs().max())
    assert float((la - lb).abs().max()) <= 1e-4


def test_step_on_full_sequence_sets_status_and_keeps_length():
    """One sequence of the batch is at capacity: its token is dropped (status bit), its length stays, the step is
    still the decode step of the cache as it is; the other sequence advances."""
    w = small(batch=2, ctx_min=16 * 10, ctx=16 * 12, decode_steps=0)
    a, b = setup(w), setup(w)
    cap = a.table.shape[1] * 16
    for d in (a, b):
        d.ckv.set_tail_mode(binding.CKV_TAIL_ON)
        d.lens[0] = cap                                  # sequence 0 fills its page table completely
        d.lens[1] = cap - 21
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, cap)
    q = torch.from_numpy(synth.queries(w, 0)).to(a.dtype).cuda()
    gen = torch.Generator().manual_seed(7)
    kn = torch.randn(w.batch, w.num_kv_heads, 128, generator=gen).to(a.dtype).cuda()
    vn = torch.randn(w.batch, w.num_kv_heads, 128, generator=gen).to(a.dtype).cuda()
    n1 = int(a.lens[1])
    oa, la, ia, ca = a.ckv.step(q, kn, vn, a.k_pool, a.v_pool, a.table, a.lens, cap, w.budget_tokens)
    b.ckv.append(b.k_pool, b.v_pool, b.table, b.lens, kn, vn)
    ob, lb, ib, cb = b.ckv.decode(q, b.k_pool, b.v_pool, b.table, b.lens, cap, w.budget_tokens)
    torch.cuda.synchronize()
    assert a.ckv.read_status() & binding.CKV_DEV_SEQ_FULL
    assert b.ckv.read_status() & binding.CKV_DEV_SEQ_FULL
    assert a.lens.cpu().tolist() == [cap, n1 + 1] and torch.equal(a.lens, b.lens)
    assert torch.equal(ia, ib) and torch.equal(ca, cb) and torch.equal(oa, ob) and torch.equal(la, lb)


def test_step_replayed_in_a_cuda_graph_advances_lengths():
    """The length hand-over inside the launch (a counter of CTAs that have read the old lengths) must leave the
    counter ready for the next replay: 12 replays of one captured step advance every length by 12."""
    w = small(ctx=16 * 30 + 7, decode_steps=12)
    a, b = setup(w), setup(w)
    for d in (a, b):
        d.ckv.set_tail_mode(binding.CKV_TAIL_ON)
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    q, kn, vn = rows(a, 0)
    max_len = a.max_len + 12
    outs = a.ckv.alloc_outputs(w.batch, w.budget_tokens)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        a.ckv.step(q, kn, vn, a.k_pool, a.v_pool, a.table, a.lens, max_len, w.budget_tokens, outs)   # warm-up, step 1
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            a.ckv.step(q, kn, vn, a.k_pool, a.v_pool, a.table, a.lens, max_len, w.budget_tokens, outs)
        for _ in range(11):
            g.replay()
    torch.cuda.synchronize()
    for _ in range(12):
        b.ckv.append(b.k_pool, b.v_pool, b.table, b.lens, kn, vn)
    ob, lb, ib, cb = b.ckv.decode(q, b.k_pool, b.v_pool, b.table, b.lens, max_len, w.budget_tokens)
    torch.cuda.synchronize()
    assert torch.equal(a.lens, b.lens)
    assert torch.equal(outs[0], ob) and torch.equal(outs[2], ib) and torch.equal(outs[3], cb)
    assert a.ckv.read_status() == 0


@pytest.mark.parametrize("seed", range(10))
def test_tail_modes_agree_on_random_shapes(seed):
    """Random small shapes (group size, block size, ragged lengths down to a single token, budgets from tiny to
    "select everything"): a few steps in tail mode and in the two-call arrangement give the same lengths, pages and
    summaries bit for bit, the same ids, and outputs within the bf16 tolerance."""
    import random
    rnd = random.Random(1000 + seed)
    hkv = rnd.choice([1, 2, 4])
    g = rnd.choice([1, 2, 4, 8])
    bs = rnd.choice([16, 16, 32, 64])
    batch = rnd.randint(1, 5)
    ctx = rnd.choice([3, 17, 16 * 5, 16 * 33 + 7, 16 * 150 + 11])
    ctx_min = rnd.choice([1, max(1, ctx // 3), ctx])
    kblocks = rnd.choice([4, 7, 30])
    steps = 5
    w = small(batch=batch, num_q_heads=hkv * g, num_kv_heads=hkv, block_size=bs, ctx_min=min(ctx_min, ctx), ctx=ctx,
              decode_steps=steps, budget_tokens=bs * kblocks, needles=0)
    a, b = setup(w), setup(w)
    a.ckv.set_tail_mode(binding.CKV_TAIL_ON)
    b.ckv.set_tail_mode(binding.CKV_TAIL_OFF)
    for d in (a, b):
        d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    for t in range(steps):
        q, kn, vn = rows(a, t)
        max_len = a.max_len + t + 1
        oa, la, ia, ca = a.ckv.step(q, kn, vn, a.k_pool, a.v_pool, a.table, a.lens, max_len, w.budget_tokens)
        ob, lb, ib, cb = b.ckv.step(q, kn, vn, b.k_pool, b.v_pool, b.table, b.lens, max_len, w.budget_tokens)
        torch.cuda.synchronize()
        assert torch.equal(a.lens, b.lens), (seed, t)
        assert torch.equal(ca, cb), (seed, t)
        sa, sb = a.ckv.copy_scores(w.batch), b.ckv.copy_scores(w.batch)
        same_ids = torch.equal(ia, ib)
        if not same_ids:   # only a near-tie at the cut may differ (the last block's terms differ by rounding)
            for s in range(w.batch):
                for h in range(hkv):
                    n = int(ca[s, h])
                    x, y = set(ia[s, h, :n].tolist()), set(ib[s, h, :n].tolist())
                    for blk in x ^ y:
                        cut = min(float(sa[s, h, i]) for i in x)
                        assert abs(float(sa[s, h, blk]) - cut) <= 1e-4 * max(cut, 1e-30), (seed, t, s, h, blk)
        else:
            scale = float(ob.float().abs().max()) + 1e-6
            assert float((oa.float() - ob.float()).abs().max()) <= 2e-2 * scale, (seed, t)
            assert float((la - lb).abs().max()) <= 1e-3, (seed, t)
    torch.cuda.synchronize()
    assert torch.equal(a.k_pool, b.k_pool) and torch.equal(a.v_pool, b.v_pool)
    for x, y in zip(a.ckv.export_stats(), b.ckv.export_stats()):
        assert torch.equal(x, y)
    assert a.ckv.read_status() == 0 and b.ckv.read_status() == 0


def test_step_with_fewer_sequences_than_the_context_allows():
    """A context sized for 5 sequences stepping 2 of them (the first two rows of every array): both arrangements."""
    w5 = small(batch=5, ctx_min=16 * 20 + 1, ctx=16 * 45 + 5, decode_steps=6)
    w2 = w5.with_(batch=2)
    for mode in (binding.CKV_TAIL_ON, binding.CKV_TAIL_OFF):
        big, ref = setup(w5), setup(w2)
        # the generator keys rows by (seed, sequence, head): the two-sequence workload is the first two sequences of
        # the five-sequence one (different pages, same contents)
        for d in (big, ref):
            d.ckv.set_tail_mode(mode)
        big.ckv.stats_build(big.k_pool, big.v_pool, big.table, big.lens, big.max_len)
        ref.ckv.stats_build(ref.k_pool, ref.v_pool, ref.table, ref.lens, ref.max_len)
        torch.cuda.synchronize()
        if not torch.equal(big.lens[:2], ref.lens):
            pytest.skip("the generator does not key sequences independently of the batch size")
        for t in range(6):
            q5, kn5, vn5 = rows(big, t)
            q2, kn2, vn2 = rows(ref, t)
            assert torch.equal(q5[:2], q2)
            ob, lb, ib, cb = big.ckv.step(q5[:2].contiguous(), kn5[:2].contiguous(), vn5[:2].contiguous(), big.k_pool,
                                          big.v_pool, big.table, big.lens, big.max_len + t + 1, w5.budget_tokens)
            orf, lr, ir, cr = ref.ckv.step(q2, kn2, vn2, ref.k_pool, ref.v_pool, ref.table, ref.lens,
                                           ref.max_len + t + 1, w2.budget_tokens)
            torch.cuda.synchronize()
            assert torch.equal(big.lens[:2], ref.lens) and int(big.lens[2]) == int(setup_len(w5, 2))
            assert torch.equal(ib, ir) and torch.equal(cb, cr)
            assert torch.equal(ob, orf) and torch.equal(lb, lr)
        assert big.ckv.read_status() == 0 and ref.ckv.read_status() == 0


def setup_len(w, s):
    return int(synth.seq_lens(w)[s])
