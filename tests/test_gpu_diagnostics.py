"""ckv_exact_blocks and the block-level diagnostics built on it, against the oracle's token-level definitions."""
import numpy as np
import pytest
import torch

from oracle import compkv_oracle as O
from paper_2609_26300_b200 import diagnostics as D
from paper_2609_26300_b200 import synth

from helpers import dev_q, setup, unit_inputs

pytestmark = pytest.mark.gpu

TOY = synth.CONFIGS[1]


def small(**kw):
    base = dict(batch=2, num_q_heads=8, num_kv_heads=2, ctx=16 * 70 + 5, budget_tokens=16 * 12, needles=4,
                outlier_dims=2, decode_steps=0, name="diag")
    base.update(kw)
    return TOY.with_(**base)


@pytest.mark.parametrize("bs", [16, 32, 64])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("hq", [2, 8, 16])   # G = 1, 4, 8
def test_exact_block_statistics_match_the_oracle(bs, dtype, hq):
    w = small(block_size=bs, num_q_heads=hq, ctx_min=16 * 20 + 3)
    d = setup(w, dtype)
    q = dev_q(d)
    logZ, zmean, zvar = d.ckv.exact_blocks(q, d.k_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    assert d.ckv.read_status() == 0
    G = w.group
    for s in range(w.batch):
        n = int(d.lens[s])
        x = -(-n // bs)
        for h in range(w.num_kv_heads):
            qq, K, _ = unit_inputs(w, s, h, n)
            rows = slice(h * G, (h + 1) * G)
            e = D.exact_unit(logZ[s, rows].cpu().numpy(), zmean[s, rows].cpu().numpy(), zvar[s, rows].cpu().numpy(), n, bs)
            assert np.all(np.isnan(logZ[s, rows, x:].cpu().numpy()))   # blocks past the end are not written
            for g in range(G):
                ref = O.exact_blocks(qq[g], K, bs)
                assert np.allclose(e.logZ[g], ref.logZ, rtol=0, atol=2e-4 * max(1.0, np.abs(ref.logZ).max()))
                assert np.allclose(e.sigma2[g], ref.sigma2, rtol=2e-3, atol=1e-5)
                assert np.allclose(e.p[g], ref.p, rtol=2e-3, atol=1e-9)
                assert np.allclose(e.rho[g], ref.rho, rtol=0, atol=5e-4 * ref.p + 1e-9)   # a difference of near-equal terms
                assert np.all(e.rho[g] >= 0.0)


def test_kl_of_a_selection_matches_the_token_level_definition():
    w = small(ctx=16 * 50 + 11)
    d = setup(w)
    d.ckv.stats_build(d.k_pool, d.v_pool, d.table, d.lens, d.max_len)
    q = dev_q(d)
    out, lse, ids, cnt = d.ckv.decode(q, d.k_pool, d.v_pool, d.table, d.lens, d.max_len, w.budget_tokens)
    scores = d.ckv.copy_scores(w.batch)
    logZ, zmean, zvar = d.ckv.exact_blocks(q, d.k_pool, d.table, d.lens, d.max_len)
    torch.cuda.synchronize()
    G, bs = w.group, w.block_size
    for s in range(w.batch):
        n = int(d.lens[s])
        for h in range(w.num_kv_heads):
            qq, K, _ = unit_inputs(w, s, h, n)
            rows = slice(h * G, (h + 1) * G)
            e = D.exact_unit(logZ[s, rows].cpu().numpy(), zmean[s, rows].cpu().numpy(), zvar[s, rows].cpu().numpy(), n, bs)
            sel = ids[s, h, :int(cnt[s, h])].cpu().numpy()
            kl_mean, kl_drop = D.kl_of_selection(e, sel), D.kl_of_selection(e, sel, drop=True)
            for g in range(G):
                P, Ph, _, _ = O.token_dists(qq[g], K, bs, sel)
                assert abs(kl_mean[g] - O.kl(Ph, P)) <= 2e-4
                P, Ph, _, _ = O.token_dists(qq[g], K, bs, sel, drop=True)
                assert abs(kl_drop[g] - O.kl(Ph, P)) <= 2e-4
                assert -1e-6 <= kl_mean[g] <= kl_drop[g] + 1e-6            # compensation never hurts (App. A.6)
            # the selection metrics are well defined and consistent
            cap = D.residual_capture(e, sel)
            best = D.residual_capture(e, D.exact_topk(e, w.budget_tokens // bs))
            assert 0.0 <= cap <= best + 1e-9 <= 1.0 + 1e-9
            rho_s = D.spearman(scores[s, h].cpu().numpy(), e)
            assert -1.0 <= rho_s <= 1.0
