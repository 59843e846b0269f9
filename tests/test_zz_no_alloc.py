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


def test_static_scratch_rejects_what_does_not_fit():
    L = binding.ckv_layout(64, 8, 128, 16, 16, 4, 1, binding.CKV_BF16, 256, 64, 1 << 16, 1, 2, 0.0)
    z = torch.zeros(256, 64, 128, dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros(4, 8, 16, 128, dtype=torch.bfloat16, device="cuda")
    table = torch.zeros(256, 64, dtype=torch.int32, device="cuda")
    lens = torch.ones(256, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.CompKVError) as e:   # 256 * 64 heads * 528 B * 64 splits > 4 MiB
        binding.dense_decode_static(L, z, pool, pool, table, lens, 16)
    assert e.value.status == binding.CKV_ERR_CAPACITY
