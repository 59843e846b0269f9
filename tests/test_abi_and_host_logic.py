"""CPU-side checks of the C ABI: the library loads, exports everything include/compkv.h declares, and
its host-only entry points (layout validation, buffer sizing) behave.  No compute call is made."""
import ctypes
import os
import re

import pytest

from paper_2609_26300_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "compkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ckv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), "libcompkv.so does not export %s" % n
    assert sorted(binding.EXPORTS) == names
    assert lib.ckv_version() >= 100


def test_strerror_names_every_status():
    seen = set()
    for st in range(0, -7, -1):
        msg = binding.strerror(st)
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 7
    assert binding.strerror(-99) == "unknown status"


def layout(**kw):
    base = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, block_size=16, page_size=16, var_groups=4,
                group_layout=1, kv_dtype=binding.CKV_BF16, max_batch=4, max_blocks_per_seq=8196, num_pages=40000,
                sink_blocks=1, recent_blocks=2, sm_scale=0.0)
    base.update(kw)
    return binding.ckv_layout(**base)


def test_sizes_follow_the_summary_layout():
    L = layout()
    stats, work = binding.query_sizes(L)
    rows = 4 * 8 * 8196
    # 2d + r fp32 scalars per block (the count is implied by the sequence length)
    assert rows * (2 * 128 + 4) * 4 <= stats <= rows * (2 * 128 + 4) * 4 + 3 * 256
    ko, do, vo = binding.stats_offsets(L)
    assert ko == 0 and do >= rows * 128 * 4 and vo >= do + rows * 4 * 4
    assert ko % 256 == do % 256 == vo % 256 == 0
    assert work > rows * 4 * 8      # at least the per-(block, head) pairs
    half, _ = binding.query_sizes(layout(stat_bf16=1))
    assert rows * (128 + 4) * 4 <= half <= rows * (128 + 4) * 4 + 3 * 256   # bf16 means: half the mean bytes
    s128, _ = binding.query_sizes(layout(var_groups=128))
    assert s128 - stats >= rows * (128 - 4) * 4 - 256


@pytest.mark.parametrize("bad", [dict(num_q_heads=24), dict(head_dim=64), dict(block_size=48), dict(page_size=32),
                                 dict(var_groups=3), dict(var_groups=96), dict(group_layout=2), dict(kv_dtype=5),
                                 dict(max_batch=0), dict(num_pages=0), dict(sink_blocks=-1),
                                 dict(sm_scale=float("nan")), dict(max_blocks_per_seq=0), dict(variant=8),
                                 dict(variant=-1), dict(stat_bf16=2), dict(stat_bf16=1, kv_dtype=binding.CKV_F32),
                                 dict(stat_bf16=1, var_groups=128),
                                 # more scan tiles per step than the kernels' index arithmetic is exact for (2^24)
                                 dict(max_batch=1 << 16, max_blocks_per_seq=1 << 21),
                                 dict(max_batch=64, max_blocks_per_seq=1 << 20)])
def test_bad_layouts_are_rejected(bad):
    with pytest.raises(binding.CompKVError) as e:
        binding.query_sizes(layout(**bad))
    assert e.value.status == binding.CKV_ERR_BAD_LAYOUT


def test_layout_just_below_the_tile_limit_is_accepted():
    # 64 sequences x 8 KV heads x (2^20 - 32) / 32 tiles = 2^24 - 512 tiles per step
    stats, work = binding.query_sizes(layout(max_batch=64, max_blocks_per_seq=(1 << 20) - 32))
    assert stats > 0 and work > 0


@pytest.mark.parametrize("ok", [dict(var_groups=1), dict(var_groups=64), dict(var_groups=128), dict(block_size=64),
                                dict(num_q_heads=64), dict(num_q_heads=8), dict(kv_dtype=binding.CKV_F32),
                                dict(variant=7), dict(variant=binding.VARIANT_DROP), dict(stat_bf16=1)])
def test_good_layouts_are_accepted(ok):
    stats, work = binding.query_sizes(layout(**ok))
    assert stats > 0 and work > 0


def test_null_arguments_are_rejected_before_any_cuda_call():
    lib = binding.load()
    L = layout()
    assert lib.ckv_query_sizes(None, None, None) == binding.CKV_ERR_INVALID_ARG
    ctx = ctypes.c_void_p(None)
    assert lib.ckv_create(ctypes.byref(L), None, 0, None, 0, None, ctypes.byref(ctx)) == binding.CKV_ERR_INVALID_ARG
    assert lib.ckv_decode(None, None, None, None, None, None, 1, 16, 64, None, None, None, None, None) \
        == binding.CKV_ERR_INVALID_ARG
    assert lib.ckv_append(None, None, None, None, None, None, None, 1, None) == binding.CKV_ERR_INVALID_ARG
    assert lib.ckv_launch_count(None) == 0
    # the entry points added after the first ones: a null context is refused before anything else is looked at
    bad = binding.CKV_ERR_INVALID_ARG
    assert lib.ckv_step(None, None, None, None, None, None, None, None, 1, 16, 64, None, None, None, None, None) == bad
    assert lib.ckv_prefill(None, None, None, None, None, None, None, None, 16, 1, 16, None) == bad
    assert lib.ckv_exact_blocks(None, None, None, None, None, 1, 16, None, None, None, None) == bad
    assert lib.ckv_scan_profile(None, None, None, 1, 16, 1, None, None) == bad
    assert lib.ckv_set_tail_mode(None, binding.CKV_TAIL_ON) == bad
    assert lib.ckv_debug_set(None, 0, 0) == bad
    assert lib.ckv_dense_decode(None, None, None, None, None, None, 1, 16, None, None, None) == bad
    assert lib.ckv_stats_build(None, None, None, None, None, 1, 16, None) == bad
    assert lib.ckv_dense_decode_static(None, None, None, None, None, None, 1, 16, None, None, None) == bad
    lib.ckv_destroy(None)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="not built"):
        binding.load()
