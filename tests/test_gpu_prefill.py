"""ckv_prefill: chunks of contiguous rows written into the paged cache with their summaries, against the cache image
and the summaries the prefill-time build produces from it."""
import numpy as np
import pytest
import torch

from paper_2609_26300_b200 import synth

from helpers import setup

pytestmark = pytest.mark.gpu

TOY = synth.CONFIGS[1]


def small(**kw):
    base = dict(batch=2, num_q_heads=8, num_kv_heads=2, ctx=16 * 40 + 11, budget_tokens=16 * 12, needles=0,
                outlier_dims=2, decode_steps=0, name="prefill")
    base.update(kw)
    return TOY.with_(**base)


def source_rows(w, dtype):
    """[batch][ctx][kv_heads][128] rows of the synthetic cache, as the projection layer would hand them over."""
    k = np.zeros((w.batch, w.ctx, w.num_kv_heads, 128), np.float32)
    v = np.zeros_like(k)
    lens = synth.seq_lens(w)
    for s in range(w.batch):
        for h in range(w.num_kv_heads):
            K, V = synth.unit_kv(w, s, h)
            k[s, :lens[s], h] = K[:lens[s]]
            v[s, :lens[s], h] = V[:lens[s]]
    return torch.from_numpy(k).to(dtype).cuda(), torch.from_numpy(v).to(dtype).cuda(), lens


@pytest.mark.parametrize("bs", [16, 32, 64])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("chunks", [(10 ** 6,), (37, 16, 1, 15, 200, 10 ** 6), (1, 1, 1, 62, 3, 10 ** 6)])
def test_chunked_prefill_equals_build(bs, dtype, chunks):
    w = small(block_size=bs, ctx_min=16 * 20 + 3)
    ref = setup(w, dtype)                                   # the cache image and the build over it
    ref.ckv.stats_build(ref.k_pool, ref.v_pool, ref.table, ref.lens, ref.max_len)
    want = [t.clone() for t in ref.ckv.export_stats(w.batch)]
    d = setup(w, dtype)
    d.k_pool.fill_(float("nan")); d.v_pool.fill_(float("nan"))
    k_src, v_src, lens = source_rows(w, dtype)
    cur = torch.zeros(w.batch, dtype=torch.int32, device="cuda")
    done = np.zeros(w.batch, np.int64)
    for c in chunks:
        new = np.minimum(c, lens - done).astype(np.int32)
        if new.max() == 0:
            break
        # every sequence's chunk starts at row 0 of its slice of the source buffer
        ks = torch.zeros(w.batch, int(new.max()), w.num_kv_heads, 128, dtype=dtype, device="cuda")
        vs = torch.zeros_like(ks)
        for s in range(w.batch):
            ks[s, :new[s]] = k_src[s, done[s]:done[s] + new[s]]
            vs[s, :new[s]] = v_src[s, done[s]:done[s] + new[s]]
        d.ckv.prefill(d.k_pool, d.v_pool, d.table, cur, ks, vs, torch.from_numpy(new).cuda(), int(new.max()))
        done += new
        torch.cuda.synchronize()
        assert np.array_equal(cur.cpu().numpy(), done)
    assert d.ckv.read_status() == 0
    assert np.array_equal(done, lens)
    got = d.ckv.export_stats(w.batch)
    for s in range(w.batch):
        n = int(lens[s]); x = -(-n // bs)
        for t in range(0, n, 16):                           # cache rows, bit for bit
            pg = int(d.table[s, t // 16]); m = min(16, n - t)
            assert torch.equal(d.k_pool[pg, :, :m], ref.k_pool[pg, :, :m])
            assert torch.equal(d.v_pool[pg, :, :m], ref.v_pool[pg, :, :m])
        for g, r in zip(got, want):                         # summaries, bit for bit
            assert torch.equal(g[s, :, :x], r[s, :, :x])


def test_prefill_then_decode_steps_and_capacity():
    w = small(ctx=16 * 30 + 5, decode_steps=4)
    ref = setup(w)
    ref.ckv.stats_build(ref.k_pool, ref.v_pool, ref.table, ref.lens, ref.max_len)
    d = setup(w)
    k_src, v_src, lens = source_rows(w, torch.bfloat16)
    cur = torch.zeros(w.batch, dtype=torch.int32, device="cuda")
    d.ckv.prefill(d.k_pool, d.v_pool, d.table, cur, k_src, v_src, torch.from_numpy(lens).cuda(), int(lens.max()))
    q = torch.from_numpy(synth.queries(w, 0)).bfloat16().cuda()
    a = d.ckv.decode(q, d.k_pool, d.v_pool, d.table, cur, d.max_len, w.budget_tokens)
    b = ref.ckv.decode(q, ref.k_pool, ref.v_pool, ref.table, ref.lens, ref.max_len, w.budget_tokens)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[2], b[2]) and torch.equal(a[3], b[3])
    # more tokens than the page table can hold: the excess is dropped and flagged
    cap = d.ckv.layout.max_blocks_per_seq * w.block_size
    room = cap - int(cur.max())
    extra = torch.full((w.batch,), room + 7, dtype=torch.int32, device="cuda")
    ks = torch.zeros(w.batch, room + 7, w.num_kv_heads, 128, dtype=torch.bfloat16, device="cuda")
    before = cur.clone()
    d.ckv.prefill(d.k_pool, d.v_pool, d.table, cur, ks, ks, extra, room + 7)
    torch.cuda.synchronize()
    assert d.ckv.read_status() & 2
    assert torch.all(cur == torch.minimum(before + room + 7, torch.full_like(cur, cap)))
