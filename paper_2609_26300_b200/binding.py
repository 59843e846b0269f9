"""Thin ctypes binding of libcompkv.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams; every step of the decode path runs in the
library's CUDA kernels.  There is no fallback: if the library has not been built, or a call
returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcompkv.so")

VARIANT_FIRST_ORDER_MASS, VARIANT_RANK_BY_MASS, VARIANT_DROP = 1, 2, 4
CKV_BF16, CKV_F32 = 0, 1
CKV_TAIL_AUTO, CKV_TAIL_OFF, CKV_TAIL_ON = 0, 1, 2
CKV_OK = 0
CKV_ERR_INVALID_ARG, CKV_ERR_BAD_LAYOUT, CKV_ERR_BUDGET_TOO_SMALL = -1, -2, -3
CKV_ERR_CAPACITY, CKV_ERR_CUDA, CKV_ERR_TIMEOUT = -4, -5, -6
CKV_DEBUG_SKIP_FILL = 1
CKV_DEV_BAD_PAGE, CKV_DEV_SEQ_FULL, CKV_DEV_NONFINITE, CKV_DEV_TIMEOUT, CKV_DEV_BAD_COPY = 1, 2, 4, 8, 16

EXPORTS = ["ckv_version", "ckv_strerror", "ckv_last_cuda_error", "ckv_query_sizes", "ckv_stats_offsets",
           "ckv_create", "ckv_destroy", "ckv_stats_build", "ckv_stats_export", "ckv_append", "ckv_prefill", "ckv_decode", "ckv_step", "ckv_decode_profile", "ckv_scan_profile", "ckv_dense_decode",
           "ckv_dense_decode_static",
           "ckv_exact_blocks", "ckv_copy_scores", "ckv_step_host", "ckv_read_status", "ckv_launch_count",
           "ckv_set_tail_mode", "ckv_debug_set"]


class ckv_layout(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block_size", ctypes.c_int32), ("page_size", ctypes.c_int32), ("var_groups", ctypes.c_int32),
                ("group_layout", ctypes.c_int32), ("kv_dtype", ctypes.c_int32), ("max_batch", ctypes.c_int32),
                ("max_blocks_per_seq", ctypes.c_int32), ("num_pages", ctypes.c_int32),
                ("sink_blocks", ctypes.c_int32), ("recent_blocks", ctypes.c_int32), ("sm_scale", ctypes.c_float),
                ("variant", ctypes.c_int32), ("stat_bf16", ctypes.c_int32)]


class CompKVError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        extra = ""
        if status == CKV_ERR_CUDA:
            extra = ", cudaError %d" % load().ckv_last_cuda_error()
        super().__init__("%s failed: %s (status %d%s)" % (what, strerror(status), status, extra))


_lib = None


def load() -> ctypes.CDLL:
    """Load libcompkv.so (built by paper_2609_26300_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libcompkv.so is not built (%s): run `python -m paper_2609_26300_b200.build`; "
                           "there is no fallback path" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lp = ctypes.POINTER(ckv_layout)
    szp = ctypes.POINTER(ctypes.c_size_t)
    lib.ckv_version.restype = i32
    lib.ckv_strerror.restype = ctypes.c_char_p
    lib.ckv_strerror.argtypes = [i32]
    lib.ckv_last_cuda_error.restype = i32
    lib.ckv_query_sizes.argtypes = [lp, szp, szp]
    lib.ckv_stats_offsets.argtypes = [lp, szp, szp, szp]
    lib.ckv_create.argtypes = [lp, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
    lib.ckv_destroy.argtypes = [vp]
    lib.ckv_destroy.restype = None
    lib.ckv_stats_build.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp]
    lib.ckv_stats_export.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.ckv_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.ckv_prefill.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp]
    lib.ckv_prefill.restype = i32
    lib.ckv_decode.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.ckv_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.ckv_decode_profile.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp,
                                       ctypes.POINTER(ctypes.c_float)]
    lib.ckv_scan_profile.argtypes = [vp, vp, vp, i32, i32, i32, vp, ctypes.POINTER(ctypes.c_float)]
    lib.ckv_dense_decode.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    lib.ckv_dense_decode_static.argtypes = [lp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    lib.ckv_dense_decode_static.restype = i32
    lib.ckv_exact_blocks.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.ckv_exact_blocks.restype = i32
    lib.ckv_copy_scores.argtypes = [vp, vp, i32, vp]
    lib.ckv_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.ckv_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
    lib.ckv_launch_count.argtypes = [vp]
    lib.ckv_launch_count.restype = ctypes.c_int64
    lib.ckv_set_tail_mode.argtypes = [vp, ctypes.c_int]
    lib.ckv_set_tail_mode.restype = ctypes.c_int
    lib.ckv_debug_set.argtypes = [vp, ctypes.c_uint32, ctypes.c_int]
    lib.ckv_debug_set.restype = ctypes.c_int
    for name in ("ckv_query_sizes", "ckv_stats_offsets", "ckv_create", "ckv_stats_build", "ckv_stats_export", "ckv_append",
                 "ckv_decode", "ckv_step", "ckv_decode_profile", "ckv_scan_profile", "ckv_dense_decode", "ckv_copy_scores", "ckv_step_host", "ckv_read_status"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().ckv_strerror(status).decode()


def _check(status: int, what: str) -> None:
    if status != CKV_OK:
        raise CompKVError(status, what)


def query_sizes(layout: ckv_layout) -> Tuple[int, int]:
    a, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load().ckv_query_sizes(ctypes.byref(layout), ctypes.byref(a), ctypes.byref(b)), "ckv_query_sizes")
    return a.value, b.value


def stats_offsets(layout: ckv_layout) -> Tuple[int, int, int]:
    a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load().ckv_stats_offsets(ctypes.byref(layout), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "ckv_stats_offsets")
    return a.value, b.value, c.value


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def dense_decode_static(layout: ckv_layout, q, k_pool, v_pool, page_table, seq_lens, max_seq_len: int, out=None,
                        lse=None):
    """ckv_dense_decode_static: dense decode attention that needs no context and no workspace.

    For callers that cannot allocate device memory for the library.  The scratch is a fixed array inside the
    library, shared by all calls: do not let two calls overlap on the GPU.  Returns (out, lse)."""
    batch = q.shape[0]
    if out is None:
        out = torch.empty(batch, layout.num_q_heads, layout.head_dim, dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty(batch, layout.num_q_heads, dtype=torch.float32, device=q.device)
    _check(load().ckv_dense_decode_static(ctypes.byref(layout), _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_table),
                                          _ptr(seq_lens), batch, int(max_seq_len), _ptr(out), _ptr(lse), _stream()),
           "ckv_dense_decode_static")
    return out, lse


class CompKV:
    """A ckv_ctx plus the two device buffers it works in (allocated with torch)."""

    def __init__(self, num_q_heads: int, num_kv_heads: int, max_batch: int, max_blocks_per_seq: int, num_pages: int,
                 block_size: int = 16, var_groups: int = 4, group_layout: int = 1, kv_dtype: int = CKV_BF16,
                 sink_blocks: int = 1, recent_blocks: int = 2, sm_scale: float = 0.0, head_dim: int = 128,
                 page_size: int = 16, device: str = "cuda", variant: int = 0, stat_bf16: int = 0):
        self.lib = load()
        self.layout = ckv_layout(num_q_heads, num_kv_heads, head_dim, block_size, page_size, var_groups,
                                 group_layout, kv_dtype, max_batch, max_blocks_per_seq, num_pages, sink_blocks,
                                 recent_blocks, sm_scale, variant, stat_bf16)
        self.stats_bytes, self.work_bytes = query_sizes(self.layout)
        self.device = torch.device(device)
        self.stats = torch.zeros(self.stats_bytes, dtype=torch.uint8, device=self.device)
        self.work = torch.zeros(self.work_bytes, dtype=torch.uint8, device=self.device)
        self.dtype = torch.bfloat16 if kv_dtype == CKV_BF16 else torch.float32
        self._ctx = ctypes.c_void_p(None)
        with torch.cuda.device(self.device):
            _check(self.lib.ckv_create(ctypes.byref(self.layout), self.stats.data_ptr(), self.stats_bytes,
                                       self.work.data_ptr(), self.work_bytes, _stream(), ctypes.byref(self._ctx)),
                   "ckv_create")

    def close(self) -> None:
        if self._ctx:
            self.lib.ckv_destroy(self._ctx)
            self._ctx = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- summaries ----------------------------------------------------------------------------------------
    def export_stats(self, batch: Optional[int] = None):
        """ckv_stats_export: (kmean, dbar, vmean) as fp32 tensors [batch][kv_heads][max_blocks][...]."""
        L = self.layout
        batch = batch or L.max_batch
        shape = (batch, L.num_kv_heads, L.max_blocks_per_seq)
        km = torch.empty(*shape, L.head_dim, dtype=torch.float32, device=self.device)
        db = torch.empty(*shape, L.var_groups, dtype=torch.float32, device=self.device)
        vm = torch.empty(*shape, L.head_dim, dtype=torch.float32, device=self.device)
        _check(self.lib.ckv_stats_export(self._ctx, batch, _ptr(km), _ptr(db), _ptr(vm), _stream()),
               "ckv_stats_export")
        return km, db, vm

    # ---- C ABI calls --------------------------------------------------------------------------------------
    def stats_build(self, k_pool, v_pool, page_table, seq_lens, max_seq_len: int) -> None:
        _check(self.lib.ckv_stats_build(self._ctx, _ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_lens),
                                        seq_lens.shape[0], int(max_seq_len), _stream()), "ckv_stats_build")

    def append(self, k_pool, v_pool, page_table, seq_lens, k_new, v_new) -> None:
        _check(self.lib.ckv_append(self._ctx, _ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_lens),
                                   _ptr(k_new), _ptr(v_new), seq_lens.shape[0], _stream()), "ckv_append")

    def alloc_outputs(self, batch: int, budget_tokens: int):
        L = self.layout
        kcap = budget_tokens // L.block_size
        out = torch.empty(batch, L.num_q_heads, L.head_dim, dtype=self.dtype, device=self.device)
        lse = torch.empty(batch, L.num_q_heads, dtype=torch.float32, device=self.device)
        ids = torch.empty(batch, L.num_kv_heads, max(kcap, 1), dtype=torch.int32, device=self.device)
        cnt = torch.empty(batch, L.num_kv_heads, dtype=torch.int32, device=self.device)
        return out, lse, ids, cnt

    def decode(self, q, k_pool, v_pool, page_table, seq_lens, max_seq_len: int, budget_tokens: int, outputs=None):
        batch = q.shape[0]
        out, lse, ids, cnt = outputs if outputs is not None else self.alloc_outputs(batch, budget_tokens)
        _check(self.lib.ckv_decode(self._ctx, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_lens),
                                   batch, int(max_seq_len), int(budget_tokens), _ptr(out), _ptr(lse), _ptr(ids),
                                   _ptr(cnt), _stream()), "ckv_decode")
        return out, lse, ids, cnt

    def prefill(self, k_pool, v_pool, page_table, seq_lens, k_src, v_src, new_lens, max_new: int) -> None:
        """ckv_prefill: k_src / v_src [batch][tokens][kv_heads][128]; new_lens int32 [batch] on the device."""
        _check(self.lib.ckv_prefill(self._ctx, _ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(seq_lens),
                                    _ptr(k_src), _ptr(v_src), _ptr(new_lens), int(k_src.shape[1]), int(k_src.shape[0]),
                                    int(max_new), _stream()), "ckv_prefill")

    def step(self, q, k_new, v_new, k_pool, v_pool, page_table, seq_lens, max_seq_len: int, budget_tokens: int,
             outputs=None):
        """ckv_step: append (k_new, v_new), then decode q; returns (out, lse, sel_ids, sel_cnt)."""
        batch = q.shape[0]
        out, lse, ids, cnt = outputs if outputs is not None else self.alloc_outputs(batch, budget_tokens)
        _check(self.lib.ckv_step(self._ctx, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool),
                                 _ptr(page_table), _ptr(seq_lens), batch, int(max_seq_len), int(budget_tokens),
                                 _ptr(out), _ptr(lse), _ptr(ids), _ptr(cnt), _stream()), "ckv_step")
        return out, lse, ids, cnt

    def decode_profile(self, q, k_pool, v_pool, page_table, seq_lens, max_seq_len: int, budget_tokens: int,
                       outputs=None):
        """ckv_decode_profile: returns (outputs, [scan, select, attention, merge] milliseconds)."""
        batch = q.shape[0]
        out, lse, ids, cnt = outputs if outputs is not None else self.alloc_outputs(batch, budget_tokens)
        ms = (ctypes.c_float * 4)()
        _check(self.lib.ckv_decode_profile(self._ctx, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_table),
                                           _ptr(seq_lens), batch, int(max_seq_len), int(budget_tokens), _ptr(out),
                                           _ptr(lse), _ptr(ids), _ptr(cnt), _stream(), ms), "ckv_decode_profile")
        return (out, lse, ids, cnt), [float(x) for x in ms]

    def scan_profile(self, q, seq_lens, max_seq_len: int, reps: int) -> float:
        """ckv_scan_profile: average milliseconds of one summary-scan launch over `reps` back-to-back launches."""
        ms = ctypes.c_float(0.0)
        _check(self.lib.ckv_scan_profile(self._ctx, _ptr(q), _ptr(seq_lens), q.shape[0], int(max_seq_len), int(reps),
                                         _stream(), ctypes.byref(ms)), "ckv_scan_profile")
        return float(ms.value)

    def dense_decode(self, q, k_pool, v_pool, page_table, seq_lens, max_seq_len: int, out=None, lse=None):
        batch = q.shape[0]
        L = self.layout
        if out is None:
            out = torch.empty(batch, L.num_q_heads, L.head_dim, dtype=self.dtype, device=self.device)
        if lse is None:
            lse = torch.empty(batch, L.num_q_heads, dtype=torch.float32, device=self.device)
        _check(self.lib.ckv_dense_decode(self._ctx, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(page_table),
                                         _ptr(seq_lens), batch, int(max_seq_len), _ptr(out), _ptr(lse), _stream()),
               "ckv_dense_decode")
        return out, lse

    def exact_blocks(self, q, k_pool, page_table, seq_lens, max_seq_len: int):
        """ckv_exact_blocks: (logZ, zmean, zvar), each fp32 [batch][q_heads][max_blocks] (blocks past the end: NaN)."""
        L = self.layout
        batch = q.shape[0]
        outs = [torch.full((batch, L.num_q_heads, L.max_blocks_per_seq), float("nan"), dtype=torch.float32,
                           device=self.device) for _ in range(3)]
        _check(self.lib.ckv_exact_blocks(self._ctx, _ptr(q), _ptr(k_pool), _ptr(page_table), _ptr(seq_lens), batch,
                                         int(max_seq_len), _ptr(outs[0]), _ptr(outs[1]), _ptr(outs[2]), _stream()),
               "ckv_exact_blocks")
        return tuple(outs)

    def copy_scores(self, batch: int) -> torch.Tensor:
        L = self.layout
        dst = torch.empty(batch, L.num_kv_heads, L.max_blocks_per_seq, dtype=torch.float32, device=self.device)
        _check(self.lib.ckv_copy_scores(self._ctx, _ptr(dst), batch, _stream()), "ckv_copy_scores")
        return dst

    def step_host(self, q_host, k_new_host, v_new_host, k_pool, v_pool, page_table, seq_lens, max_seq_len: int,
                  budget_tokens: int, out_host, sel_ids_host, sel_cnt_host) -> None:
        """Host tensors (pinned) in and out; the device pools, page table and seq_lens stay on the GPU."""
        for t in (q_host, k_new_host, v_new_host, out_host, sel_ids_host, sel_cnt_host):
            assert not t.is_cuda
        _check(self.lib.ckv_step_host(self._ctx, _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), _ptr(k_pool),
                                      _ptr(v_pool), _ptr(page_table), _ptr(seq_lens), q_host.shape[0],
                                      int(max_seq_len), int(budget_tokens), _ptr(out_host), _ptr(sel_ids_host),
                                      _ptr(sel_cnt_host), _stream()), "ckv_step_host")

    def read_status(self) -> int:
        st = ctypes.c_int32(0)
        _check(self.lib.ckv_read_status(self._ctx, ctypes.byref(st), _stream()), "ckv_read_status")
        return st.value

    def launch_count(self) -> int:
        return int(self.lib.ckv_launch_count(self._ctx))

    def set_tail_mode(self, mode: int) -> None:
        """ckv_set_tail_mode: CKV_TAIL_AUTO (default), CKV_TAIL_OFF, CKV_TAIL_ON."""
        _check(self.lib.ckv_set_tail_mode(self._ctx, int(mode)), "ckv_set_tail_mode")

    def debug_set(self, spin_limit: int = 0, flags: int = 0) -> None:
        """ckv_debug_set (test hook): polls a bounded device-side wait makes (0 = default), CKV_DEBUG_* flags."""
        _check(self.lib.ckv_debug_set(self._ctx, int(spin_limit), int(flags)), "ckv_debug_set")
