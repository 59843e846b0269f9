"""ckv_dense_decode_static: the entry point for hosts that cannot give the library device memory (no context,
no workspace; its scratch is a fixed array inside the library).  Called through the C ABI and compared with
ckv_dense_decode on the same inputs, twice in a row: the second call finds the first call's partials and status
word in the shared array and must not be disturbed by them.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import compkv_oracle as O
from paper_2609_26300_b200 import binding, synth

from helpers import OUT_TOL, dev_q, rel_inf, setup, unit_inputs

pytestmark = pytest.mark.gpu


def test_static_scratch_dense_decode_matches_the_workspace_version_twice():
    base = synth.CONFIGS[1].with_(batch=3, num_q_heads=8, num_kv_heads=2, ctx_min=16 * 40 + 3, ctx=16 * 300 + 9,
                                  decode_steps=0, needles=4, outlier_dims=2, name="no_alloc")
    for call, w in enumerate((base, base.with_(seed=base.seed + 17))):   # two calls in a row, different data
        d = setup(w)
        q = dev_q(d)
        ref, ref_lse = d.ckv.dense_decode(q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
        torch.cuda.synchronize()
        out, lse = binding.dense_decode_static(d.ckv.layout, q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
        torch.cuda.synchronize()
        tol = OUT_TOL[d.dtype]
        assert rel_inf(out.double().cpu().numpy(), ref.double().cpu().numpy()) <= tol
        assert float((lse - ref_lse).abs().max()) <= 1e-4
        # and against the oracle, for one unit, so that a shared mistake would not hide
        G = w.group
        qq, K, V = unit_inputs(w, 1, 1, int(d.lens[1]))
        assert rel_inf(out[1, G:2 * G].double().cpu().numpy(), O.dense(qq, K, V)[0]) <= tol


@pytest.mark.parametrize("hq,hkv,dtype", [(2, 2, torch.bfloat16), (16, 2, torch.bfloat16), (4, 2, torch.float32),
                                          (8, 2, torch.float32)])
def test_static_entry_without_any_context_for_its_layout(hq, hkv, dtype):
    """The callers this entry point is for never create a context, so nothing has set the attributes of the kernels
    their layout needs: the entry point has to do that itself, for every (group size, page type) it meets, not only
    for the first one it sees on a device.  Group sizes 1, 8, 2 and 4 in turn, bf16 and fp32 pages (the fp32 layout
    merges in a launch of its own), no ckv_create anywhere in this test; each result against the oracle's dense
    attention."""
    w = synth.CONFIGS[1].with_(batch=2, num_q_heads=hq, num_kv_heads=hkv, ctx_min=16 * 30 + 5, ctx=16 * 90 + 11,
                               decode_steps=0, needles=2, outlier_dims=2, name="no_ctx")
    k_pool, v_pool, table, lens = synth.make_pools(w, dtype=dtype)
    max_blocks = synth.pages_per_seq(w)
    L = binding.ckv_layout(hq, hkv, 128, 16, 16, 4, 1, binding.CKV_BF16 if dtype == torch.bfloat16 else binding.CKV_F32,
                           w.batch, max_blocks, k_pool.shape[0], 1, 2, 0.0, 0, 0)
    k_pool, v_pool, table, lens = (t.cuda() for t in (k_pool, v_pool, table, lens))
    q = torch.from_numpy(synth.queries(w, 0)).to(dtype).cuda()
    for _ in range(2):   # two calls in a row: the second finds the first one's partials and counters in the array
        out, lse = binding.dense_decode_static(L, q, k_pool, v_pool, table, lens, int(lens.max()))
        torch.cuda.synchronize()
        G = w.group
        for s in range(w.batch):
            for h in range(hkv):
                qq, K, V = unit_inputs(w, s, h, int(lens[s]))
                ref, ref_lse = O.dense(qq, K, V)
                assert rel_inf(out[s, h * G:(h + 1) * G].double().cpu().numpy(), ref) <= OUT_TOL[dtype]
                assert np.abs(lse[s, h * G:(h + 1) * G].double().cpu().numpy() - ref_lse).max() <= 1e-4 * max(1.0, np.abs(ref_lse).max())


def test_static_scratch_rejects_what_does_not_fit():
    L = binding.ckv_layout(64, 8, 128, 16, 16, 4, 1, binding.CKV_BF16, 256, 64, 1 << 16, 1, 2, 0.0)
    z = torch.zeros(256, 64, 128, dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros(4, 8, 16, 128, dtype=torch.bfloat16, device="cuda")
    table = torch.zeros(256, 64, dtype=torch.int32, device="cuda")
    lens = torch.ones(256, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CompKVError) as e:   # 256 * 64 heads * 528 B * 64 splits > 4 MiB
        binding.dense_decode_static(L, z, pool, pool, table, lens, 16)
    assert e.value.status == binding.CKV_ERR_CAPACITY
    # the second limit: one split counter per unit, 192 of them
    L2 = binding.ckv_layout(8, 8, 128, 16, 16, 4, 1, binding.CKV_BF16, 25, 64, 1 << 16, 1, 2, 0.0)
    z2 = torch.zeros(25, 8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.CompKVError) as e:   # 25 * 8 = 200 units > 192
        binding.dense_decode_static(L2, z2, pool, pool, table, lens, 16)
    assert e.value.status == binding.CKV_ERR_CAPACITY
