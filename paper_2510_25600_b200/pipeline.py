"""One pass of the PureKV hot path over a batch: the sequence of C-ABI calls a caller makes.

    layers <= CLIE layer : dense causal prefill; the CLIE layer also yields the window scores C
    higher layers        : ST-SpAttn prefill
    then                 : V-norm weighting + top-h selection and K/V compaction of the
                           compressed layers

This module only sequences calls of `binding` and owns the device buffers (torch); it does
no arithmetic of the method.  `run_host` is the end-to-end form: inputs start in pinned host
memory and the compact cache is read back to the host.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as P


class PureKVPipeline:
    def __init__(self, seq_lens: Sequence[int], n_prefix: Sequence[int], n_frames: Sequence[int], mask,
                 n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: torch.dtype,
                 scored_layers: Sequence[int], compacted_layers: Sequence[int], window: int, keep_ratio: float,
                 kv_layers: Optional[int] = None):
        """`mask` has the STMask attributes.  Layers up to max(scored_layers) run dense causal attention,
        the rest ST-SpAttn.  K/V exist for kv_layers >= n_layers layers (default n_layers)."""
        self.mask, self.n_layers = mask, n_layers
        self.h, self.hkv, self.d, self.dtype = n_q_heads, n_kv_heads, head_dim, dtype
        self.code = P.BF16 if dtype == torch.bfloat16 else P.FP32
        self.clie = max(scored_layers)
        self.scored = tuple(scored_layers)
        self.compacted = tuple(compacted_layers)
        assert self.compacted == tuple(range(self.compacted[0], self.compacted[-1] + 1)), "compacted layers must be contiguous"
        self.kv_layers = kv_layers if kv_layers is not None else max(n_layers, self.compacted[-1] + 1)
        self.window, self.keep_ratio = window, keep_ratio
        self.batch = P.Batch(seq_lens, n_prefix, n_frames)
        self.budget = P.Budget(self.batch, window, keep_ratio)
        t = self.batch.total_tokens
        dev = "cuda"
        params_dense = P.st_params(mask)
        params_dense.flags |= P.FLAG_DENSE_CAUSAL
        self.params_dense, self.params_st = params_dense, P.st_params(mask)
        hh = (n_q_heads, n_kv_heads)
        self.plan_buf_dense = torch.empty(max(1, P.purekv_plan_bytes(self.batch, params_dense, self.code, head_dim, *hh)),
                                          dtype=torch.uint8, device=dev)
        self.plan_buf_st = torch.empty(max(1, P.purekv_plan_bytes(self.batch, self.params_st, self.code, head_dim, *hh)),
                                       dtype=torch.uint8, device=dev)
        self.prefill_ws = None
        self._h_plans = [(torch.empty(self.plan_buf_dense.numel(), dtype=torch.uint8, pin_memory=True),
                          torch.empty(self.plan_buf_st.numel(), dtype=torch.uint8, pin_memory=True)) for _ in range(3)]
        self._h_plan_events = [None] * len(self._h_plans)
        self._plan_slot = 0
        self.o = torch.empty((n_layers, t, n_q_heads, head_dim), dtype=dtype, device=dev)
        self.c = torch.empty((len(self.scored), n_kv_heads, t), dtype=torch.float32, device=dev)
        # one-pass tensor-core scores where the entry point supports the shape (bf16, head_dim 128, window and any
        # clipped window a multiple of 8); the two-pass kernels otherwise
        self.one_pass_scores = (dtype == torch.bfloat16 and head_dim == 128 and window % 8 == 0 and
                                all(l >= window or l % 8 == 0 for l in seq_lens))
        self.lse = torch.empty((len(self.scored), n_q_heads, t), dtype=torch.float32, device=dev)
        self.score_ws = torch.empty(P.purekv_score_ws_bytes(self.batch, window, n_q_heads), dtype=torch.uint8, device=dev)
        nc = len(self.compacted)
        self.select_ws = torch.empty(P.purekv_select_ws_bytes(self.batch, nc, n_kv_heads), dtype=torch.uint8, device=dev)
        self.idx = torch.empty((nc, n_kv_heads, self.budget.total_kept), dtype=torch.int32, device=dev)
        self.k_c = torch.empty((nc, self.budget.total_kept, n_kv_heads, head_dim), dtype=dtype, device=dev)
        self.v_c = torch.empty_like(self.k_c)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.plan_dense = self.plan_st = None
        # prefill per layer, score (1 kernel one-pass, 3 otherwise), select (2), compact
        self.launches_per_step = n_layers + (1 if self.one_pass_scores else 3) * len(self.scored) + 2 + 1

    def build_plans(self) -> None:
        """Plans both masks on the host into pinned buffers and enqueues their copies on the current stream without
        waiting, so planning overlaps the GPU work already in flight.  A small ring of pinned buffers keeps a plan
        alive until its copy has run."""
        slot = self._plan_slot
        self._plan_slot = (slot + 1) % len(self._h_plans)
        if self._h_plan_events[slot] is not None:
            self._h_plan_events[slot].synchronize()
        plans = []
        for params, h_buf, d_buf in ((self.params_dense, self._h_plans[slot][0], self.plan_buf_dense),
                                     (self.params_st, self._h_plans[slot][1], self.plan_buf_st)):
            h_used, info = P.purekv_plan_build_host(self.batch, params, self.code, self.d, self.h, self.hkv, out=h_buf)
            d_buf[:info.bytes_used].copy_(h_used, non_blocking=True)
            plans.append(P.Plan(d_buf, info))
        ev = torch.cuda.Event()
        ev.record()
        self._h_plan_events[slot] = ev
        self.plan_dense, self.plan_st = plans
        need = max(16, self.plan_dense.info.ws_bytes, self.plan_st.info.ws_bytes)
        if self.prefill_ws is None or self.prefill_ws.numel() < need:
            self.prefill_ws = torch.empty(need, dtype=torch.uint8, device="cuda")

    def prefill_layer(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> None:
        plan = self.plan_dense if layer <= self.clie else self.plan_st
        # a scored layer is dense causal: its prefill also leaves the rows' log-sum-exp for the one-pass scores
        lse = self.lse[self.scored.index(layer)] if (self.one_pass_scores and layer in self.scored) else None
        P.purekv_st_sparse_prefill(q, k, v, self.batch, plan, out=self.o[layer], lse=lse, status=self.status,
                                   ws=self.prefill_ws)

    def run_device(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, events=None, marks=None) -> None:
        """q [n_layers,T,H,d], k,v [kv_layers,T,H_kv,d] on the GPU.  Results in self.o / idx / k_c / v_c.
        `events`, if given, is a list of (start, end) torch.cuda.Event pairs, one per prefill launch (an event
        between two launches keeps the second from starting under the first's tail); `marks`, if given, is three
        events recorded before the first prefill launch, after the last dense-causal one and after the last one."""
        self.build_plans()
        if marks is not None:
            marks[0].record()
        for layer in range(self.n_layers):
            if events is not None:
                events[layer][0].record()
            self.prefill_layer(layer, q[layer], k[layer], v[layer])
            if events is not None:
                events[layer][1].record()
            if marks is not None and layer == self.clie:
                marks[1].record()
        if marks is not None:
            marks[2].record()
        for n, layer in enumerate(self.scored):
            if self.one_pass_scores:
                P.purekv_lowlayer_score_lse(q[layer], k[layer], self.lse[n], self.batch, self.window, c_out=self.c[n],
                                            status=self.status)
            else:
                P.purekv_lowlayer_score(q[layer], k[layer], self.batch, self.window, c_out=self.c[n], ws=self.score_ws)
        lo, hi = self.compacted[0], self.compacted[-1] + 1
        P.purekv_select_topk(self.c[len(self.scored) - 1], v[lo:hi], self.batch, self.budget, idx_out=self.idx,
                             ws=self.select_ws)
        P.purekv_compact_kv(k[lo:hi], v[lo:hi], self.idx, self.batch, self.budget, k_out=self.k_c, v_out=self.v_c)

    def alloc_host_io(self):
        """Pinned host buffers for run_host: (q, k, v) inputs and (k_c, v_c, o_last) outputs."""
        t = self.batch.total_tokens
        pin = dict(dtype=self.dtype, pin_memory=True)
        ins = (torch.empty((self.n_layers, t, self.h, self.d), **pin),
               torch.empty((self.kv_layers, t, self.hkv, self.d), **pin),
               torch.empty((self.kv_layers, t, self.hkv, self.d), **pin))
        outs = (torch.empty(tuple(self.k_c.shape), **pin), torch.empty(tuple(self.v_c.shape), **pin),
                torch.empty((t, self.h, self.d), **pin))
        return ins, outs

    def run_host(self, h_in, h_out, d_in) -> None:
        """End to end: pinned host Q/K/V -> device (d_in, caller-owned staging) -> hot path -> compact cache and
        the last layer's O back in pinned host memory.  Synchronises before returning."""
        for src, dst in zip(h_in, d_in):
            dst.copy_(src, non_blocking=True)
        self.run_device(*d_in)
        h_out[0].copy_(self.k_c, non_blocking=True)
        h_out[1].copy_(self.v_c, non_blocking=True)
        h_out[2].copy_(self.o[self.n_layers - 1], non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def check_status(self) -> None:
        P.purekv_poll_status(self.status)
