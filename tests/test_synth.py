"""The synthetic input generator: determinism, shapes, and the structure the recipe promises."""
import numpy as np
import torch

from paper_2609_26300_b200 import synth


def test_units_are_deterministic_and_bf16_exact():
    w = synth.CONFIGS[1]
    k1, v1 = synth.unit_kv(w, 0, 0)
    k2, v2 = synth.unit_kv(w, 0, 0)
    assert np.array_equal(k1, k2) and np.array_equal(v1, v2)
    assert k1.shape == (w.ctx + w.decode_steps, w.head_dim) and k1.dtype == np.float32
    back = torch.from_numpy(k1).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back, k1)
    q = synth.queries(w)
    assert q.shape == (1, 4, 128)
    assert np.array_equal(torch.from_numpy(q).to(torch.bfloat16).float().numpy(), q)


def test_round_bf16_matches_torch():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 37.0
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).float().numpy()
    assert np.array_equal(synth.round_bf16_(x.copy()), ref)


def test_needles_raise_group_mean_logit_by_six():
    w = synth.CONFIGS[1]
    k, _ = synth.unit_kv(w, 0, 0, with_tail=False)
    q = synth.queries(w)[0]
    pos = synth.needle_positions(w, 0, 0, w.ctx)
    assert len(pos) == 8 and pos.min() >= 16 and pos.max() < w.ctx - 32
    z = (q.astype(np.float64) @ k.T.astype(np.float64)) / np.sqrt(128)
    zm = z.mean(0)
    others = np.delete(zm, pos)
    assert abs(zm[pos].mean() - 6.0) < 1.0 and abs(others.mean()) < 0.2


def test_noise_levels_per_16_token_unit():
    w = synth.CONFIGS[1].with_(needles=0)
    k, _ = synth.unit_kv(w, 0, 0, with_tail=False)
    std = k.reshape(-1, 16, 128).std(axis=1).mean(axis=1)
    nearest = np.abs(std[:, None] / synth.NOISE_LEVELS[None, :] - 1).min(1)
    assert np.all(nearest < 0.25)
    assert len(np.unique(np.abs(std[:, None] / synth.NOISE_LEVELS[None, :] - 1).argmin(1))) == 3


def test_outlier_channels_scaled():
    w = synth.CONFIGS[2].with_(ctx=2048, needles=0)
    k, _ = synth.unit_kv(w, 0, 3, with_tail=False)
    ch = synth.outlier_channels(w, 0, 3)
    assert len(ch) == 4
    rms = np.sqrt((k.astype(np.float64) ** 2).mean(0))
    rest = np.delete(rms, ch)
    assert np.all(rms[ch] > 5 * rest.mean())


def test_ragged_lengths_and_page_table():
    w = synth.CONFIGS[4]
    lens = synth.seq_lens(w)
    assert lens.shape == (16,) and lens.min() >= 16384 and lens.max() <= 65536
    table, total = synth.page_table(w)
    used = table[table >= 0]
    assert len(used) == total and len(np.unique(used)) == total
    need = -(-(lens.astype(np.int64) + w.decode_steps) // 16)
    assert np.array_equal((table >= 0).sum(1), need)
    assert not np.array_equal(table[0, :8], np.arange(8))      # shuffled


def test_pools_hold_the_units_and_tail_rows():
    w = synth.CONFIGS[1].with_(ctx=100, decode_steps=5, num_kv_heads=2, num_q_heads=4, needles=0)
    k_pool, v_pool, table, lens = synth.make_pools(w, dtype=torch.float32, threads=1)
    for h in range(2):
        k, v = synth.unit_kv(w, 0, h)
        assert k.shape[0] == 105
        pages = table[0, :7].long()
        got = k_pool[pages, h].reshape(-1, 128)[:105].numpy()
        assert np.array_equal(got, k)
        kt, vt = synth.unit_tail(w, 0, h)
        assert np.array_equal(kt, k[100:]) and np.array_equal(vt, v[100:])
    kn, vn = synth.appended_rows(w, 2)
    assert np.array_equal(kn[0, 1], synth.unit_kv(w, 0, 1)[0][102])
    assert int(lens[0]) == 100
