"""Host plumbing that drives the C-ABI library over a synthetic workload.

Allocates device memory with torch, feeds the seeded raw tensors through
ippd_append_kv (context and question tokens: the stand-in for prefill) and runs
decode steps through ippd_begin_step / ippd_append_kv(STEP) / ippd_decode_attention.
No attention arithmetic happens here.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .workloads import Workload


class Runner:
    def __init__(self, wl: Workload, device: str = "cuda:0", out_dtype: int = B.BF16, kernel: int = 0,
                 layers_per_call: Optional[int] = None, tiles_per_split: int = 0, branch_align: int = B.TILE_TOKENS,
                 fused: bool = True, kv_dtype: int = B.KV_BF16):
        if not torch.cuda.is_available():
            raise RuntimeError("the IPPD library needs a CUDA device; there is no CPU fallback")
        self.wl = wl
        self.fused = fused  # one ippd_decode_step call per layer group instead of append_kv(STEP) + decode_attention
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        g = wl.geom
        self.geom = B.make_geometry(g.n_layers, g.n_q_heads, g.n_kv_heads, g.head_dim, g.rope_theta,
                                    branch_align, out_dtype)
        self.layout = B.Layout(self.geom, wl.ctx_len, wl.q_count, wl.q_len, wl.max_new, shared_len=wl.shared_len)
        if kernel:
            self.layout.set_option(B.OPT_KERNEL, kernel)
        self.kv_dtype = kv_dtype
        if kv_dtype != B.KV_BF16:
            self.layout.set_option(B.OPT_KV_DTYPE, kv_dtype)  # before the cache is sized and bound
        if layers_per_call:
            self.layout.set_option(B.OPT_LAYERS_PER_CALL, layers_per_call)
        if tiles_per_split:
            self.layout.set_option(B.OPT_TILES_PER_SPLIT, tiles_per_split)
        self.layers_per_call = layers_per_call or g.n_layers
        nbytes, _ = self.layout.cache_bytes()
        self.cache = self.alloc_bytes(nbytes, "cache")
        self.stream = torch.cuda.current_stream(self.device).cuda_stream
        self.layout.bind_cache(self.cache, self.stream)
        self.workspace = self.alloc_bytes(self.layout.workspace_bytes(self.layers_per_call), "workspace")
        self.out_torch_dtype = torch.float32 if out_dtype == B.F32 else torch.bfloat16

    def alloc_bytes(self, nbytes: int, what: str) -> torch.Tensor:
        """Device buffer handed to the library (uint8, 256-byte aligned).  Subclasses may surround it with guard bands."""
        return torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    def alloc_out(self, n_active: int) -> torch.Tensor:
        g = self.wl.geom
        shape = (g.n_layers, n_active, g.n_q_heads, g.head_dim)
        n = int(np.prod(shape)) * (4 if self.out_torch_dtype == torch.float32 else 2)
        return self.alloc_bytes(n, "out").view(self.out_torch_dtype).view(shape)

    # ------------------------------------------------------------------ prefill stand-in
    def load_header(self, prompts: Optional[Sequence[int]] = None):
        """Appends the context and question tokens of the given prompts (default all), layer by layer."""
        wl, g = self.wl, self.wl.geom
        prompts = list(range(wl.n_prompts)) if prompts is None else list(prompts)
        qids = [k for b in prompts for k in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1]))]
        for layer in range(g.n_layers):
            if wl.shared_len > 0:
                k, v = wl.shared_kv(layer, self.device)
                self.layout.append_kv(layer, 1, B.APPEND_SHARED, None, k, v, self.stream)
            for b in prompts:
                if wl.ctx_len[b] == 0:
                    continue
                k, v = wl.ctx_kv(b, layer, self.device)
                self.layout.append_kv(layer, 1, B.APPEND_CONTEXT, [b], k, v, self.stream)
            ks, vs = zip(*[wl.question_kv(k, layer, self.device) for k in qids])
            self.layout.append_kv(layer, 1, B.APPEND_QUESTION, qids, torch.cat(ks).contiguous(),
                                  torch.cat(vs).contiguous(), self.stream)
        torch.cuda.synchronize(self.device)

    def header_inputs(self, layer: int):
        """Raw q, k, v of every header token at one layer, in the order of the layout's hdr_* tables (the shared
        instruction, then per prompt its context tokens and its questions' tokens): [n_hdr, H, D] each."""
        wl, dev = self.wl, self.device
        qs, ks, vs = [], [], []
        if wl.shared_len > 0:
            k, v = wl.shared_kv(layer, dev)
            qs.append(wl.shared_q(layer, dev)); ks.append(k); vs.append(v)
        for b in range(wl.n_prompts):
            if wl.ctx_len[b] > 0:
                k, v = wl.ctx_kv(b, layer, dev)
                qs.append(wl.ctx_q(b, layer, dev)); ks.append(k); vs.append(v)
            for qid in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1])):
                k, v = wl.question_kv(qid, layer, dev)
                qs.append(wl.question_q(qid, layer, dev)); ks.append(k); vs.append(v)
        return torch.cat(qs).contiguous(), torch.cat(ks).contiguous(), torch.cat(vs).contiguous()

    def prefill(self, layers_per_call: int = 1, keep_out: bool = True):
        """Prefill of the stacked header through ippd_prefill_attention, `layers_per_call` layers per call: fills the
        cache with the header's K/V and returns the attention output of every header token,
        [n_layers, n_hdr, Hq, D] (None when keep_out is False)."""
        g = self.wl.geom
        need = self.layout.workspace_bytes(layers_per_call)
        if need > self.workspace.numel():
            self.workspace = self.alloc_bytes(need, "workspace")
        outs = []
        for l0 in range(0, g.n_layers, layers_per_call):
            n = min(layers_per_call, g.n_layers - l0)
            qkv = [self.header_inputs(l) for l in range(l0, l0 + n)]
            q = torch.stack([t[0] for t in qkv]).contiguous()
            k = torch.stack([t[1] for t in qkv]).contiguous()
            v = torch.stack([t[2] for t in qkv]).contiguous()
            shape = (n, q.shape[1], g.n_q_heads, g.head_dim)
            nbytes = int(np.prod(shape)) * (4 if self.out_torch_dtype == torch.float32 else 2)
            out = self.alloc_bytes(nbytes, "out").view(self.out_torch_dtype).view(shape)
            self.layout.prefill_attention(l0, n, q, k, v, out, self.workspace, self.stream)
            torch.cuda.synchronize(self.device)
            if keep_out:
                outs.append(out)
        return torch.cat(outs) if keep_out else None

    # ------------------------------------------------------------------ decode
    def step_inputs(self, s: int, act: np.ndarray):
        """Raw q, k, v of step s for the active questions, all layers: [layers, A, H, D] each."""
        wl, g = self.wl, self.wl.geom
        q = torch.stack([wl.step_q(s, l, act, self.device) for l in range(g.n_layers)])
        kv = [wl.step_kv(s, l, act, self.device) for l in range(g.n_layers)]
        k = torch.stack([a for a, _ in kv])
        v = torch.stack([b for _, b in kv])
        return q.contiguous(), k.contiguous(), v.contiguous()

    def decode_step(self, act: np.ndarray, answer_idx: np.ndarray, q, k, v, out=None):
        """One decode step over all layers, in groups of `layers_per_call` layers."""
        g = self.wl.geom
        A = len(act)
        if out is None:
            out = self.alloc_out(A)
        self.layout.begin_step(act, answer_idx, self.stream)
        if A == 0:
            return out
        lpc = self.layers_per_call
        if self.fused:
            self.layout.decode_step_grouped(lpc, q, k, v, out, self.workspace, self.stream)
            return out
        for l0 in range(0, g.n_layers, lpc):
            n = min(lpc, g.n_layers - l0)
            self.layout.append_kv(l0, n, B.APPEND_STEP, None, k[l0:l0 + n], v[l0:l0 + n], self.stream)
            self.layout.decode_attention(l0, n, q[l0:l0 + n], out[l0:l0 + n], self.workspace, self.stream)
        return out

    def set_layers_per_call(self, n: int):
        """Changes the number of layers per launch (the next begin_step plans for it; the workspace is re-sized)."""
        self.layout.set_option(B.OPT_LAYERS_PER_CALL, n)
        self.layers_per_call = n
        need = self.layout.workspace_bytes(n)
        if need > self.workspace.numel():
            self.workspace = self.alloc_bytes(need, "workspace")

    def append_all_steps(self, layers_per_chunk: int = 8):
        """Writes the K/V of EVERY decode step of the schedule into the cache (a step's slot depends only on the
        question and the step index), so that afterwards any step can be run in any order."""
        wl, g = self.wl, self.wl.geom
        for s in range(wl.n_steps):
            act = wl.active(s)
            if len(act) == 0:
                continue
            self.layout.begin_step(act, np.full(len(act), s, dtype=np.int32), self.stream)
            for l0 in range(0, g.n_layers, layers_per_chunk):
                n = min(layers_per_chunk, g.n_layers - l0)
                kv = [wl.step_kv(s, l, act, self.device) for l in range(l0, l0 + n)]
                k = torch.stack([a for a, _ in kv]).contiguous()
                v = torch.stack([b for _, b in kv]).contiguous()
                self.layout.append_kv(l0, n, B.APPEND_STEP, None, k, v, self.stream)
            torch.cuda.synchronize(self.device)

    def run_step(self, s: int):
        """Generates the inputs of workload step s and runs it; returns (active ids, out)."""
        act = self.wl.active(s)
        q, k, v = self.step_inputs(s, act)
        out = self.decode_step(act, np.full(len(act), s, dtype=np.int32), q, k, v)
        return act, out

    def check(self):
        w = self.layout.poll_status()
        if w:
            raise RuntimeError(f"device error word {w}")
