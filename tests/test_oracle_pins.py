"""Pins for the CPU oracle: every check compares it with something other than itself --
a library routine, a closed form, an identity the paper proves, a value the paper
prints, or brute force on tiny inputs.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import compkv_oracle as O

D = 128
RNG = np.random.default_rng(20260926)


def bf16(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def make_unit(n, g=4, d=D, noise=0.3, bs=16, seed=0):
    r = np.random.default_rng(seed)
    nb = -(-n // bs)
    c = r.standard_normal((nb, 1, d))
    k = (c + noise * r.standard_normal((nb, bs, d))).reshape(nb * bs, d)[:n]
    v = r.standard_normal((n, d))
    q = r.standard_normal((g, d))
    return bf16(q), bf16(k), bf16(v)


def golden():
    out = {}
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


# ---- dense: a library attention routine ------------------------------------------------------

@pytest.mark.parametrize("n,g", [(1, 1), (37, 4), (500, 8)])
def test_dense_matches_library_attention(n, g):
    q, k, v = make_unit(n, g, seed=n)
    out, lse = O.dense(q, k, v)
    tq, tk, tv = (torch.from_numpy(a).double() for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None])[0].numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)
    ref_lse = torch.logsumexp(tq @ tk.T / np.sqrt(D), dim=1).numpy()
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-12)


def test_dense_custom_scale():
    q, k, v = make_unit(50, 2, seed=3)
    out, _ = O.dense(q, k, v, scale=0.25)
    tq, tk, tv = (torch.from_numpy(a).double() for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], scale=0.25)[0].numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)


# ---- stats: numpy mean / population variance -------------------------------------------------

def groups_literal(d, r, layout):
    """Coordinate groups written out from the paper's wording (App. A.4), not from the oracle."""
    if r == d:
        return [[i] for i in range(d)]
    if layout == 0:   # pairs (2p, 2p+1): consecutive pairs == consecutive coordinates
        pairs = [(2 * p, 2 * p + 1) for p in range(d // 2)]
    else:             # pairs (p, p + d/2)
        pairs = [(p, p + d // 2) for p in range(d // 2)]
    per = len(pairs) // r
    return [sorted(c for pr in pairs[t * per:(t + 1) * per] for c in pr) for t in range(r)]


@pytest.mark.parametrize("bs,n", [(16, 16 * 7), (16, 16 * 5 + 3), (32, 100), (64, 65), (16, 1)])
@pytest.mark.parametrize("r,layout", [(4, 1), (4, 0), (1, 1), (64, 1), (128, 0), (16, 0)])
def test_stats_match_numpy(bs, n, r, layout):
    _, k, v = make_unit(n, 1, bs=bs, seed=bs + n)
    st = O.stats(k, v, bs, r, layout)
    grp = groups_literal(D, r, layout)
    x = -(-n // bs)
    assert len(st.cnt) == x
    for b in range(x):
        kb = k[b * bs:(b + 1) * bs].astype(np.float64)
        vb = v[b * bs:(b + 1) * bs].astype(np.float64)
        assert st.cnt[b] == len(kb)
        np.testing.assert_allclose(st.kmean[b], kb.mean(0), rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(st.vmean[b], vb.mean(0), rtol=1e-13, atol=1e-14)
        var = np.var(kb, axis=0)  # population variance
        ref = np.array([var[g].mean() for g in grp])
        np.testing.assert_allclose(st.Dbar[b], ref, rtol=1e-11, atol=1e-15)


def test_group_map_example_half_split_r4():
    # reading fixed for this build: pair p = (p, p + 64); group 0 holds pairs 0..15
    assert [O.group_of(i, 128, 4, 1) for i in (0, 15, 16, 63, 64, 79, 80, 127)] == [0, 0, 1, 3, 0, 0, 1, 3]
    assert [O.group_of(i, 128, 4, 0) for i in (0, 31, 32, 127)] == [0, 0, 1, 3]
    assert [O.group_of(i, 128, 128, 1) for i in (0, 77, 127)] == [0, 77, 127]


def test_single_token_block_has_zero_variance():
    _, k, v = make_unit(33, 1, seed=5)
    st = O.stats(k, v, 16)
    assert st.cnt[-1] == 1 and np.all(st.Dbar[-1] == 0.0)
    np.testing.assert_array_equal(st.kmean[-1], k[32].astype(np.float64))


def test_summary_size_matches_paper():
    g = golden()
    _, k, v = make_unit(64, 1, seed=1)
    st4, st128 = O.stats(k, v, 16, 4), O.stats(k, v, 16, 128)
    per_block = 1 + st4.kmean.shape[1] + st4.Dbar.shape[1] + st4.vmean.shape[1]
    assert per_block == g["summary_scalars_d128_r4"]
    assert st4.Dbar.shape[1] / st128.Dbar.shape[1] == g["variance_metadata_ratio_r4_over_r128"]


def test_append_equals_rebuild():
    _, k, v = make_unit(16 * 6 + 40, 1, seed=9)
    n0 = 16 * 6 - 1          # starts one short of a full block: covers fill, rollover, 1-token block
    for bs in (16, 32):
        st = O.stats(k[:n0], v[:n0], bs)
        for n in range(n0 + 1, len(k) + 1):
            st = O.append(st, k[:n], v[:n])
            ref = O.stats(k[:n], v[:n], bs)
            for a, b in ((st.cnt, ref.cnt), (st.kmean, ref.kmean), (st.Dbar, ref.Dbar), (st.vmean, ref.vmean)):
                np.testing.assert_array_equal(a, b)


# ---- compensated attention: special cases and the token-level definition ------------------------

def test_select_all_is_dense():
    q, k, v = make_unit(16 * 9 + 5, 4, seed=11)
    st = O.stats(k, v, 16)
    out, lse = O.sparse(q, k, v, st, np.arange(10))
    ref, ref_lse = O.dense(q, k, v)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-13)


def test_block_size_one_makes_compensation_exact():
    q, k, v = make_unit(40, 4, seed=12)
    st = O.stats(k, v, 1)
    ref, ref_lse = O.dense(q, k, v)
    for ids in ([0, 38, 39], [0, 5, 6, 7, 39], []):
        out, lse = O.sparse(q, k, v, st, ids)
        np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(lse, ref_lse, rtol=1e-12)


def test_constant_key_blocks_make_compensation_exact_for_lse():
    # identical keys inside each block => every logit equals the block mean => shared normaliser is exact,
    # and with identical values too the output is exact.
    r = np.random.default_rng(13)
    nb, bs = 9, 16
    kc = bf16(r.standard_normal((nb, 1, D))).repeat(bs, 1).reshape(nb * bs, D)
    vc = bf16(r.standard_normal((nb, 1, D))).repeat(bs, 1).reshape(nb * bs, D)
    vfree = bf16(r.standard_normal((nb * bs, D)))
    q = bf16(r.standard_normal((4, D)))
    n = nb * bs - 5
    st = O.stats(kc[:n], vc[:n], bs)
    ref, ref_lse = O.dense(q, kc[:n], vc[:n])
    out, lse = O.sparse(q, kc[:n], vc[:n], st, [0, 7, 8])
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-12)
    # values free: block weights are still exact, so the output is sum_b p_b * mean(v_b) on unselected blocks,
    # which for constant weights inside a block equals dense attention as well
    st2 = O.stats(kc[:n], vfree[:n], bs)
    ref2, _ = O.dense(q, kc[:n], vfree[:n])
    out2, _ = O.sparse(q, kc[:n], vfree[:n], st2, [0, 7, 8])
    np.testing.assert_allclose(out2, ref2, rtol=1e-11, atol=1e-12)
    assert np.all(st.Dbar == 0.0)


@pytest.mark.parametrize("bs,n", [(16, 16 * 12 + 7), (32, 32 * 6)])
def test_sparse_equals_token_level_definition(bs, n):
    """Eq. 12 must equal sum_j Phat_j * (v_j if selected else mean value of j's block), Phat from Eq. 1."""
    q, k, v = make_unit(n, 3, noise=1.0, bs=bs, seed=n)
    st = O.stats(k, v, bs)
    x = len(st.cnt)
    ids = [0, 3, 4, x - 2, x - 1]
    out, lse = O.sparse(q, k, v, st, ids)
    vsub = v.astype(np.float64).copy()
    for b in range(x):
        if b not in ids:
            vsub[b * bs:(b + 1) * bs] = v[b * bs:(b + 1) * bs].astype(np.float64).mean(0)
    for g in range(3):
        P, Ph, logD, logDh = O.token_dists(q[g], k, bs, ids)
        np.testing.assert_allclose(out[g], Ph @ vsub, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lse[g], logDh, rtol=1e-12)
        # and the token distributions themselves against a library softmax
        z = (k.astype(np.float64) @ q[g].astype(np.float64)) / np.sqrt(D)
        np.testing.assert_allclose(P, scipy.special.softmax(z), rtol=1e-11, atol=1e-300)
        zh = z.copy()
        for b in range(x):
            if b not in ids:
                zh[b * bs:(b + 1) * bs] = z[b * bs:(b + 1) * bs].mean()
        np.testing.assert_allclose(Ph, scipy.special.softmax(zh), rtol=1e-11, atol=1e-300)


def test_drop_variant_is_attention_over_selected_tokens():
    q, k, v = make_unit(16 * 8, 2, noise=1.0, seed=21)
    st = O.stats(k, v, 16)
    ids = [0, 2, 6, 7]
    rows = np.concatenate([np.arange(b * 16, b * 16 + 16) for b in ids])
    out, lse = O.sparse(q, k, v, st, ids, drop=True)
    ref, ref_lse = O.dense(q, k[rows], v[rows])
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-13)


def test_output_in_convex_hull():
    q, k, v = make_unit(16 * 20, 4, noise=1.0, seed=22)
    st = O.stats(k, v, 16)
    out, _ = O.sparse(q, k, v, st, [0, 5, 18, 19])
    lo = np.minimum(v.min(0), st.vmean.min(0)); hi = np.maximum(v.max(0), st.vmean.max(0))
    assert np.all(out >= lo - 1e-12) and np.all(out <= hi + 1e-12)


# ---- KL identities (Eq. 4, App. A.1, App. A.5) ------------------------------------------------------

def test_kl_equals_log_partition_gap_and_residual_form():
    q, k, v = make_unit(16 * 14 + 9, 4, noise=1.0, seed=31)
    ids = [0, 4, 9, 13, 14]
    x = 15
    for g in range(4):
        P, Ph, logD, logDh = O.token_dists(q[g], k, 16, ids)
        kl_def = scipy.stats.entropy(Ph, P)          # library KL(Phat || P), by definition
        assert kl_def > 1e-4
        np.testing.assert_allclose(O.kl(Ph, P), kl_def, rtol=1e-10)
        np.testing.assert_allclose(logD - logDh, kl_def, rtol=1e-9)
        eb = O.exact_blocks(q[g], k, 16)
        R = sum(eb.rho[b] for b in range(x) if b not in ids)
        np.testing.assert_allclose(-np.log1p(-R), kl_def, rtol=1e-9)
        np.testing.assert_allclose(eb.p.sum(), 1.0, rtol=1e-13)


def test_mean_vs_drop_ordering():
    q, k, v = make_unit(16 * 14, 2, noise=1.0, seed=32)
    ids = [0, 3, 12, 13]
    for g in range(2):
        P, Ph, _, _ = O.token_dists(q[g], k, 16, ids)
        Pd, Phd, logD, logDd = O.token_dists(q[g], k, 16, ids, drop=True)
        eb = O.exact_blocks(q[g], k, 16)
        kl_mean, kl_drop = scipy.stats.entropy(Ph, P), scipy.stats.entropy(Phd, Pd)
        assert 0.0 < kl_mean < kl_drop
        np.testing.assert_allclose(kl_drop, -np.log(sum(eb.p[b] for b in ids)), rtol=1e-10)
        assert np.all(eb.ratio >= 1.0 - 1e-14)   # |b| e^{zbar} <= Z_b (Jensen)


def test_second_order_expansion_of_block_ratio():
    """Z_b / (|b| e^{zbar}) = 1 + sigma^2/2 + O(sigma^3): the remainder must shrink like eps^3."""
    r = np.random.default_rng(33)
    c = r.standard_normal((6, 1, D)); e = r.standard_normal((6, 16, D)); q = r.standard_normal(D)
    rem = []
    for eps in (0.4, 0.2, 0.1):
        k = (c + eps * e).reshape(96, D).astype(np.float32)
        eb = O.exact_blocks(q.astype(np.float32), k, 16)
        rem.append(np.abs(eb.ratio - 1.0 - 0.5 * eb.sigma2).max())
        assert rem[-1] < 0.2 * (0.5 * eb.sigma2).max()    # the sigma^2/2 term itself is far bigger
    assert 5.0 < rem[0] / rem[1] < 12.0 and 5.0 < rem[1] / rem[2] < 12.0   # ~ 2^3


def test_logit_variance_is_projected_key_covariance():
    q, k, _ = make_unit(16 * 5, 1, noise=1.0, seed=34)
    eb = O.exact_blocks(q[0], k, 16)
    for b in range(5):
        cov = np.cov(k[b * 16:(b + 1) * 16].astype(np.float64).T, bias=True)
        np.testing.assert_allclose(eb.sigma2[b], q[0].astype(np.float64) @ cov @ q[0] / D, rtol=1e-9)
        z = k[b * 16:(b + 1) * 16].astype(np.float64) @ q[0] / np.sqrt(D)
        np.testing.assert_allclose(eb.sigma2[b], np.var(z), rtol=1e-9)


# ---- scorer (Eq. 8-10) ---------------------------------------------------------------------------------

def one_coordinate_unit(eps, coord, g=2, nb=8, seed=41, flat_q_group=None):
    """Keys whose within-block variation lies along one coordinate: the covariance is diagonal."""
    r = np.random.default_rng(seed)
    c = r.standard_normal((nb, 1, D))
    e = np.zeros((nb, 16, D)); e[:, :, coord] = r.standard_normal((nb, 16))
    k = (c + eps * e).reshape(nb * 16, D).astype(np.float32)
    q = r.standard_normal((g, D)).astype(np.float32)
    if flat_q_group is not None:
        q[:, flat_q_group] = np.sign(q[:, flat_q_group]) * 0.75
    return q, k, r.standard_normal((nb * 16, D)).astype(np.float32)


def test_grouped_variance_exact_when_covariance_is_diagonal_and_flat():
    # r = d: one coordinate per group, variation along one coordinate => sigma_hat^2 == sigma^2
    q, k, v = one_coordinate_unit(0.5, coord=37)
    sc = O.scores(q, O.stats(k, v, 16, r=128))
    for g in range(2):
        np.testing.assert_allclose(sc.sigma2[g], O.exact_blocks(q[g], k, 16).sigma2, rtol=1e-9)
    # r < d is NOT exact in general ...
    sc4 = O.scores(q, O.stats(k, v, 16, r=4, layout=1))
    assert np.abs(sc4.sigma2[0] / O.exact_blocks(q[0], k, 16).sigma2 - 1).max() > 0.05
    # ... unless |q_i| is constant inside the group that holds the varying coordinate
    for layout in (0, 1):
        grp = groups_literal(D, 4, layout)
        members = next(g_ for g_ in grp if 37 in g_)
        q2, k2, v2 = one_coordinate_unit(0.5, coord=37, flat_q_group=members)
        s = O.scores(q2, O.stats(k2, v2, 16, r=4, layout=layout))
        np.testing.assert_allclose(s.sigma2[1], O.exact_blocks(q2[1], k2, 16).sigma2, rtol=1e-9)


def test_mass_estimate_exact_for_constant_key_blocks_and_sums_to_one():
    r = np.random.default_rng(42)
    nb = 7
    k = bf16(r.standard_normal((nb, 1, D))).repeat(16, 1).reshape(nb * 16, D)[:nb * 16 - 6]
    v = bf16(r.standard_normal((len(k), D))); q = bf16(r.standard_normal((4, D)))
    sc = O.scores(q, O.stats(k, v, 16))
    for g in range(4):
        np.testing.assert_allclose(sc.phat[g], O.exact_blocks(q[g], k, 16).p, rtol=1e-10)
        np.testing.assert_allclose(sc.phat[g].sum(), 1.0, rtol=1e-13)
    assert np.all(sc.S == 0.0)


def test_mass_estimate_tracks_log_partition_to_third_order():
    """log Z_b = log|b| + zbar + sigma^2/2 + O(sigma^3) (App. A.2): with sigma_hat^2 == sigma^2 the
    log-ratios of phat between blocks must match the exact ones up to an eps^3 remainder."""
    rem, first = [], []
    for eps in (0.8, 0.4, 0.2):
        q, k, v = one_coordinate_unit(eps, coord=5, g=1, seed=43)
        st = O.stats(k, v, 16, r=128)
        eb = O.exact_blocks(q[0], k, 16)
        for order, store in ((2, rem), (1, first)):
            sc = O.scores(q, st, mass_order=order)
            lr = np.log(sc.phat[0]) - np.log(sc.phat[0][0])
            store.append(np.abs(lr - (eb.logZ - eb.logZ[0])).max())
    assert 5.0 < rem[0] / rem[1] < 12.0 and 5.0 < rem[1] / rem[2] < 12.0     # third order
    assert 3.0 < first[0] / first[1] < 5.0                                    # without sigma^2/2: second order
    assert rem[2] < 0.1 * first[2]


def test_first_order_mass_is_softmax_of_mean_logits():
    q, k, v = make_unit(16 * 6 + 3, 2, noise=1.0, seed=44)
    st = O.stats(k, v, 16)
    sc = O.scores(q, st, mass_order=1, outer_var=0)
    for g in range(2):
        zbar = st.kmean @ q[g].astype(np.float64) / np.sqrt(D)
        np.testing.assert_allclose(sc.zbar[g], zbar, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(sc.phat[g], scipy.special.softmax(np.log(st.cnt) + zbar), rtol=1e-11)
    np.testing.assert_allclose(sc.S, sc.phat.sum(0), rtol=1e-12)


def test_score_approaches_oracle_rule_in_small_variance_regime():
    """Eq. 10 estimates sum_g p sigma^2 (Eq. 7): with exact variance the relative gap is O(eps)."""
    gaps = []
    for eps in (0.2, 0.1):
        q, k, v = one_coordinate_unit(eps, coord=90, g=2, seed=45)
        sc = O.scores(q, O.stats(k, v, 16, r=128))
        exact = sum(O.exact_blocks(q[g], k, 16).p * O.exact_blocks(q[g], k, 16).sigma2 for g in range(2))
        gaps.append(np.abs(sc.S / exact - 1).max())
    assert gaps[0] < 0.05 and gaps[1] < gaps[0]



def test_grouped_variance_follows_the_logit_scale():
    """Eq. 8's 1/d is the squared logit scale (App. A.4 derives it from z - zbar = q (k - kbar)^T / sqrt(d)): at any
    other scale s the statistic must still equal the exact logit variance in the case where Eq. 8 is exact (r = d,
    within-block variation along one coordinate), i.e. sigma_hat^2 = s^2 sum_t w_t Dbar_t, and zbar scales with s."""
    q, k, v = one_coordinate_unit(0.5, coord=77, g=3, seed=46)
    st = O.stats(k, v, 16, r=128)
    for s in (0.25, 1.0 / np.sqrt(D) * 3.0, 0.011):
        sc = O.scores(q, st, scale=s)
        for g in range(3):
            eb = O.exact_blocks(q[g], k, 16, scale=s)
            np.testing.assert_allclose(sc.sigma2[g], eb.sigma2, rtol=1e-9)
            np.testing.assert_allclose(sc.zbar[g], st.kmean @ q[g].astype(np.float64) * s, rtol=1e-12, atol=1e-14)
    # the scale really enters squared: sigma_hat^2(2 s) = 4 sigma_hat^2(s)
    a, b = O.scores(q, st, scale=0.07), O.scores(q, st, scale=0.14)
    np.testing.assert_allclose(b.sigma2, 4.0 * a.sigma2, rtol=1e-12)


def test_block_score_closed_form_two_token_blocks():
    """Eq. 9-10 by hand.  Blocks of two tokens k = c_b +- delta_b e_{i_b}: the mean key is c_b, the only non-zero
    variance is delta_b^2 along i_b, so for head g (a = q_{g,i_b} delta_b scale)
        zbar = q_g . c_b scale,  sigma_hat^2 = a^2  (r = d)  or  scale^2 w_{g,t} delta_b^2 / |G_t|  (r = 4),
        l = log 2 + zbar + sigma_hat^2 / 2,  phat = softmax_b(l),  S_b = sum_g phat_{g,b} sigma_hat^2_{g,b},
    and the exact block sum is Z_b = 2 e^{zbar} cosh(a).  All values are dyadic, so the summaries are exact."""
    import math
    r = np.random.default_rng(47)
    nb, G = 6, 3
    c = r.integers(-12, 13, size=(nb, D)) / 8.0
    q = r.integers(-16, 17, size=(G, D)) / 16.0
    coord = [3, 40, 64, 99, 127, 17]
    delta = [0.5, 0.25, 1.0, 0.75, 0.125, 0.5]
    k = np.zeros((2 * nb, D), np.float32)
    for b in range(nb):
        e = np.zeros(D); e[coord[b]] = delta[b]
        k[2 * b], k[2 * b + 1] = c[b] + e, c[b] - e
    v = r.standard_normal((2 * nb, D)).astype(np.float32)
    scale = 1.0 / math.sqrt(D)
    for rr, layout in ((128, 1), (4, 0), (4, 1)):
        st = O.stats(k, v, 2, r=rr, layout=layout)
        sc = O.scores(q.astype(np.float32), st)
        zbar = [[sum(q[g, i] * c[b, i] for i in range(D)) * scale for b in range(nb)] for g in range(G)]
        sig = [[0.0] * nb for _ in range(G)]
        for g in range(G):
            for b in range(nb):
                if rr == 128:
                    sig[g][b] = (q[g, coord[b]] * delta[b] * scale) ** 2
                else:
                    members = next(m for m in groups_literal(D, 4, layout) if coord[b] in m)
                    w = sum(q[g, i] ** 2 for i in members)
                    sig[g][b] = scale ** 2 * w * delta[b] ** 2 / len(members)
        S = [0.0] * nb
        for g in range(G):
            ell = [math.log(2.0) + zbar[g][b] + 0.5 * sig[g][b] for b in range(nb)]
            m = max(ell)
            den = sum(math.exp(x - m) for x in ell)
            for b in range(nb):
                ph = math.exp(ell[b] - m) / den
                assert abs(sc.phat[g][b] - ph) <= 1e-12 * ph
                assert abs(sc.sigma2[g][b] - sig[g][b]) <= 1e-12 * max(sig[g][b], 1e-300)
                assert abs(sc.zbar[g][b] - zbar[g][b]) <= 1e-12 * max(abs(zbar[g][b]), 1.0)
                S[b] += ph * sig[g][b]
            if rr == 128:   # the exact block sums of the same construction
                eb = O.exact_blocks(q[g].astype(np.float32), k, 2)
                for b in range(nb):
                    a = q[g, coord[b]] * delta[b] * scale
                    assert abs(eb.logZ[b] - (math.log(2.0) + zbar[g][b] + math.log(math.cosh(a)))) <= 1e-12
        for b in range(nb):
            assert abs(sc.S[b] - S[b]) <= 1e-12 * S[b]
        # a head index or a mass taken from the wrong head must change S: the heads' terms differ
        assert max(abs(sc.phat[0][b] * sc.sigma2[0][b] - sc.phat[1][b] * sc.sigma2[1][b]) / S[b] for b in range(nb)) > 1e-3

def test_scores_invariances():
    q, k, v = make_unit(16 * 10 + 4, 4, noise=0.3, seed=46)
    st = O.stats(k, v, 16)
    sc = O.scores(q, st)
    assert np.all(sc.S >= 0.0)
    np.testing.assert_allclose(sc.phat.sum(1), 1.0, rtol=1e-13)
    # permuting tokens inside a block changes nothing
    perm = np.arange(len(k)); perm[16:32] = perm[16:32][::-1]; perm[48:64] = np.roll(perm[48:64], 3)
    st_p = O.stats(k[perm], v[perm], 16)
    np.testing.assert_allclose(O.scores(q, st_p).S, sc.S, rtol=1e-10)
    out, _ = O.sparse(q, k, v, st, [0, 1, 3, 9, 10])
    out_p, _ = O.sparse(q, k[perm], v[perm], st_p, [0, 1, 3, 9, 10])
    np.testing.assert_allclose(out_p, out, rtol=1e-9, atol=1e-12)
    # adding one constant vector to every key shifts all logits of a head equally
    shift = np.float32(0.5) * np.ones(D, np.float32)
    st_s = O.stats(k + shift, v, 16)
    np.testing.assert_allclose(st_s.Dbar, st.Dbar, rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(O.scores(q, st_s).S, sc.S, rtol=1e-6)


def test_grouped_variance_scale_statistical():
    """Isotropic noise of std s: E[Dbar_t] = s^2 (|b|-1)/|b|, so sigma_hat^2 ~ s^2 |q|^2/d (|b|-1)/|b|."""
    r = np.random.default_rng(47)
    s, nb, bs = 0.7, 400, 16
    k = (r.standard_normal((nb, 1, D)) + s * r.standard_normal((nb, bs, D))).reshape(nb * bs, D).astype(np.float32)
    q = r.standard_normal((1, D)).astype(np.float32)
    st = O.stats(k, np.zeros_like(k), bs)
    expect = s * s * (bs - 1) / bs
    # per-group mean over blocks: 32 coords x 16 tokens x 400 blocks of chi-square terms => ~0.3 % spread
    np.testing.assert_allclose(st.Dbar.mean(0), expect, rtol=0.02)
    sc = O.scores(q, st)
    np.testing.assert_allclose(sc.sigma2[0].mean(), expect * float(q[0].astype(np.float64) @ q[0]) / D, rtol=0.02)


# ---- selection (Eq. 11) ------------------------------------------------------------------------------

def brute_select(S, K, sink=1, recent=2):
    x = len(S)
    if K >= x:
        return list(range(x))
    F = {b for b in range(x) if b < sink or b >= x - recent}
    rest = sorted((b for b in range(x) if b not in F), key=lambda b: (-S[b], b))
    return sorted(F | set(rest[:K - len(F)]))


def test_select_with_other_mandatory_counts_matches_brute_force():
    """Eq. 11 with sink and recent counts other than (1, 2), 0 included, on sequences short enough for the two
    mandatory ends to overlap ("counting any overlap once")."""
    r = np.random.default_rng(52)
    seen = set()
    for trial in range(1500):
        sink, recent = int(r.integers(0, 4)), int(r.integers(0, 4))
        x = int(r.integers(1, 14))
        S = r.choice([0.0, 0.5, 1.0, 2.0], size=x) if trial % 3 == 0 else r.random(x)
        K = int(r.integers(1, 16))
        F = {b for b in range(x) if b < sink or b >= x - recent}
        if K < x and K < len(F):
            with pytest.raises(ValueError):
                O.select(S, K, sink, recent)
            continue
        ids = list(O.select(S, K, sink, recent))
        assert ids == brute_select(S, K, sink, recent), (sink, recent, x, K)
        assert len(ids) == min(K, x) and ids == sorted(set(ids))
        if K < x:
            assert F <= set(ids)
        seen.add((sink, recent, sink + recent > x))
    assert len({(a, b) for a, b, _ in seen}) == 16 and any(o for _, _, o in seen)


def test_select_matches_brute_force_with_ties():
    r = np.random.default_rng(51)
    for trial in range(300):
        x = int(r.integers(1, 40))
        S = r.choice([0.0, 0.25, 0.5, 1.0, 2.0], size=x) if trial % 2 else r.random(x)
        K = int(r.integers(3, 45))
        ids = O.select(S, K)
        assert list(ids) == brute_select(S, K)
        assert len(ids) == min(K, x) and len(set(ids)) == len(ids) and list(ids) == sorted(ids)
        for f in (0, x - 1, max(x - 2, 0)):
            assert f in ids


def test_select_budget_arithmetic_from_paper():
    g = golden()
    K = 512 // int(g["block_size"])
    assert K == g["budget512_blocks"]
    S = RNG.random(2048)
    ids = O.select(S, K, int(g["sink_blocks"]), int(g["recent_blocks"]))
    mandatory = {0, 2046, 2047}
    assert len(ids) == K and len(set(ids) - mandatory) == g["budget512_ranked_blocks"]
    with pytest.raises(ValueError):
        O.select(S, 2)


def test_single_head_exact_objective_is_solved_by_residual_ranking():
    """For G = 1 the exact objective (Eq. 2 via Eq. 4) is monotone in the sum of omitted residuals,
    so exhaustive search over subsets must pick the blocks with the largest exact residual."""
    q, k, v = make_unit(16 * 9, 1, noise=1.0, seed=52)
    x, K = 9, 4
    eb = O.exact_blocks(q[0], k, 16)
    best, best_kl = None, np.inf
    for sub in itertools.combinations(range(x), K):
        P, Ph, _, _ = O.token_dists(q[0], k, 16, list(sub))
        val = scipy.stats.entropy(Ph, P)
        if val < best_kl:
            best, best_kl = sub, val
    assert set(best) == set(np.argsort(-eb.rho)[:K])


# ---- whole decode step of a unit ------------------------------------------------------------------------

def test_decode_unit_shapes_and_select_all_limit():
    q, k, v = make_unit(16 * 6 + 2, 4, seed=61)
    st = O.stats(k, v, 16)
    out, lse, ids, sc = O.decode_unit(q, k, v, st, budget_tokens=16 * 7)
    ref, ref_lse = O.dense(q, k, v)
    assert list(ids) == list(range(7))
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    out2, _, ids2, _ = O.decode_unit(q, k, v, st, budget_tokens=16 * 4)
    assert len(ids2) == 4 and not np.allclose(out2, ref, rtol=1e-6)
