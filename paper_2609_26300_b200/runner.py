"""One decode step (ckv_step: append + decode) captured as a CUDA graph over static input buffers.

Launch plumbing only: the graph holds the library's own kernel launches; per-step inputs are copied
into the static buffers before each replay.  bench.py and the full-size parity tests share it so
that they time and check the same launch configuration.
"""
from __future__ import annotations

import torch


class GraphStep:
    def __init__(self, ckv, k_pool, v_pool, table, lens, max_len: int, budget_tokens: int, batch: int):
        L = ckv.layout
        dev, dt = ckv.device, ckv.dtype
        self.ckv = ckv
        self.q = torch.zeros(batch, L.num_q_heads, L.head_dim, dtype=dt, device=dev)
        self.k_new = torch.zeros(batch, L.num_kv_heads, L.head_dim, dtype=dt, device=dev)
        self.v_new = torch.zeros_like(self.k_new)
        self.outputs = ckv.alloc_outputs(batch, budget_tokens)
        before = ckv.launch_count()
        self.graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(self.graph):   # capture only records the launches; nothing runs here
            ckv.step(self.q, self.k_new, self.v_new, k_pool, v_pool, table, lens, max_len, budget_tokens, self.outputs)
        self.launches_per_step = ckv.launch_count() - before

    def set_inputs(self, q, k_new, v_new) -> None:
        self.q.copy_(q)
        self.k_new.copy_(k_new)
        self.v_new.copy_(v_new)

    def replay(self):
        """Runs one step on the current stream; returns (out, lse, sel_ids, sel_cnt) (static tensors)."""
        self.graph.replay()
        return self.outputs
