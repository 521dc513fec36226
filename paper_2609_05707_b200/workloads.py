"""Seeded synthetic IPPD workloads: shapes and raw q/k/v values.

This module is the only code shared by the CUDA path's harness and the CPU
oracle's harness.  It holds no attention, RoPE, mask or layout arithmetic: it
only draws lengths and tensor values.  Everything is a pure function of a
64-bit seed, so any slice of any tensor can be regenerated anywhere (host or
device) without storing it.

Value recipe.  Every raw q, k, v element is a bf16 number drawn from N(0,1):
a 64-bit counter (tensor stream id, flat element index) is hashed with a
splitmix64-style finaliser; the top 16 bits pick one of 65536 equiprobable
bins of the standard normal, whose midpoint quantile (computed in fp64) is
rounded to bf16.  The hash uses integer ops only, so the CPU and a CUDA device
produce identical bits.

Shape recipe.  Five configurations mirror the paper's common-context QA
workloads (Table "dataset statistics": 3.5-30 questions per context, questions
of 12-72 tokens, contexts of 0.2k-12k tokens, short answers): one long shared
context per prompt, many short questions, one token emitted per question per
decode step, optional per-question stop steps.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _to_i64(x: int) -> int:
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def mix64_int(x: int) -> int:
    """splitmix64 finaliser on a python int (reference for the tensor version)."""
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    # logical shift right on int64 two's-complement bits
    return (x >> n) & ((1 << (64 - n)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor (bits interpreted as uint64)."""
    x = x ^ _lsr(x, 30)
    x = x * _to_i64(_C1)
    x = x ^ _lsr(x, 27)
    x = x * _to_i64(_C2)
    x = x ^ _lsr(x, 31)
    return x


_TABLES: Dict[str, torch.Tensor] = {}


def normal_table(device="cpu") -> torch.Tensor:
    """65536 bf16 midpoint quantiles of N(0,1), built in fp64."""
    key = str(device)
    if key not in _TABLES:
        if "cpu" not in _TABLES:
            p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
            _TABLES["cpu"] = torch.special.ndtri(p).to(torch.bfloat16)
        _TABLES[key] = _TABLES["cpu"].to(device)
    return _TABLES[key]


# tensor stream kinds
K_CTX, V_CTX, K_QST, V_QST, Q_STEP, K_STEP, V_STEP, K_SHR, V_SHR, Q_CTX, Q_QST, Q_SHR = 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12


def stream_id(kind: int, index: int) -> int:
    assert 0 <= index < (1 << 20) and 0 < kind < 16
    return (kind << 20) | index


def values_at(seed: int, stream: int, flat_index: torch.Tensor) -> torch.Tensor:
    """bf16 N(0,1) values at the given flat element indices of one tensor stream."""
    assert flat_index.dtype == torch.int64
    base = _to_i64(mix64_int((seed * _GOLD + stream) & _M64))
    h = mix64(flat_index + base)
    bins = _lsr(h, 48)
    return normal_table(flat_index.device)[bins]


def values(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return values_at(seed, stream, idx)


def _randint(seed: int, tag: int, i: int, lo: int, hi: int) -> int:
    """Uniform integer in [lo, hi] (inclusive) from the counter hash."""
    h = mix64_int((seed * _GOLD + (tag << 32) + i) & _M64)
    return lo + (mix64_int(h) >> 11) % (hi - lo + 1)


@dataclass
class Geometry:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:  # K+V, bf16, one layer
        return self.n_kv_heads * self.head_dim * 2 * 2


@dataclass
class Workload:
    """One synthetic batch of stacked prompts and its decode schedule."""
    name: str
    geom: Geometry
    seed: int
    ctx_len: np.ndarray      # [B] int32
    q_count: np.ndarray      # [B] int32
    q_len: np.ndarray        # [NQ] int32
    stop: np.ndarray         # [NQ] int32: question k is active at steps 0..stop[k]-1
    max_new: np.ndarray      # [NQ] int32: branch capacity in answer tokens
    n_steps: int
    shared_len: int = 0      # tokens of an instruction shared by every prompt of the batch (0 = none)
    q_begin: np.ndarray = field(init=False)
    prompt_of: np.ndarray = field(init=False)

    def __post_init__(self):
        self.q_begin = np.zeros(len(self.q_count) + 1, dtype=np.int64)
        self.q_begin[1:] = np.cumsum(self.q_count)
        self.prompt_of = np.repeat(np.arange(len(self.q_count)), self.q_count).astype(np.int32)

    @property
    def n_prompts(self) -> int:
        return len(self.ctx_len)

    @property
    def n_questions(self) -> int:
        return len(self.q_len)

    def active(self, s: int) -> np.ndarray:
        """Sorted global ids of the questions taking part in decode step s."""
        return np.nonzero(self.stop > s)[0].astype(np.int32)

    def question_tokens(self) -> int:
        return int(sum(len(self.active(s)) for s in range(self.n_steps)))

    # ---- algorithmic bytes / flops of one decode step over all layers ----
    def step_bytes(self, s: int, kv_elem_bytes: int = 2) -> Dict[str, int]:
        """Algorithmic bytes of step s (all layers); kv_elem_bytes = 1 for the 8-bit cache variant."""
        g = self.geom
        act = self.active(s)
        kvb = g.kv_bytes_per_token * kv_elem_bytes // 2
        prompts = np.unique(self.prompt_of[act])
        # the shared instruction is read once for the whole batch, a context once per prompt with an active question
        ctx = (int(self.ctx_len[prompts].astype(np.int64).sum()) + (self.shared_len if len(act) else 0)) * kvb
        br = int((self.q_len[act].astype(np.int64) + s + 1).sum()) * kvb
        qo = len(act) * g.n_q_heads * g.head_dim * 2 * 2
        return {"context": ctx * g.n_layers, "branch": br * g.n_layers, "q_out": qo * g.n_layers,
                "total": (ctx + br + qo) * g.n_layers}

    def step_flops(self, s: int) -> int:
        g = self.geom
        act = self.active(s)
        keys = (self.shared_len + self.ctx_len[self.prompt_of[act]].astype(np.int64) + self.q_len[act] + s + 1).sum()
        return int(4 * g.head_dim * g.n_q_heads * keys) * g.n_layers

    # ---- raw tensors (bf16), generated on the requested device ----
    def _gen(self, kind: int, index: int, shape, start_row: int, device) -> torch.Tensor:
        inner = int(np.prod(shape[1:]))
        n = int(shape[0]) * inner
        return values(self.seed, stream_id(kind, index), start_row * inner, n, device).view(*shape)

    def ctx_kv(self, b: int, layer: int, device="cpu", t0: int = 0, t1: Optional[int] = None):
        """Raw (pre-RoPE) K and V of prompt b's context tokens [t0, t1) at one layer: [t, Hkv, D]."""
        g = self.geom
        L = int(self.ctx_len[b])
        t1 = L if t1 is None else t1
        shape = (t1 - t0, g.n_kv_heads, g.head_dim)
        row0 = layer * L + t0
        return (self._gen(K_CTX, b, shape, row0, device), self._gen(V_CTX, b, shape, row0, device))

    def shared_kv(self, layer: int, device="cpu"):
        """Raw K and V of the shared instruction's tokens at one layer: [shared_len, Hkv, D]."""
        g = self.geom
        shape = (self.shared_len, g.n_kv_heads, g.head_dim)
        row0 = layer * self.shared_len
        return (self._gen(K_SHR, 0, shape, row0, device), self._gen(V_SHR, 0, shape, row0, device))

    def question_kv(self, k: int, layer: int, device="cpu"):
        """Raw K and V of question k's own tokens at one layer: [n_k, Hkv, D]."""
        g = self.geom
        n = int(self.q_len[k])
        shape = (n, g.n_kv_heads, g.head_dim)
        return (self._gen(K_QST, k, shape, layer * n, device), self._gen(V_QST, k, shape, layer * n, device))

    # ---- raw queries of the header tokens (prefill) ----
    def shared_q(self, layer: int, device="cpu") -> torch.Tensor:
        """Raw queries of the shared instruction's tokens at one layer: [shared_len, Hq, D]."""
        g = self.geom
        return self._gen(Q_SHR, 0, (self.shared_len, g.n_q_heads, g.head_dim), layer * self.shared_len, device)

    def ctx_q(self, b: int, layer: int, device="cpu") -> torch.Tensor:
        """Raw queries of prompt b's context tokens at one layer: [L_b, Hq, D]."""
        g = self.geom
        L = int(self.ctx_len[b])
        return self._gen(Q_CTX, b, (L, g.n_q_heads, g.head_dim), layer * L, device)

    def question_q(self, k: int, layer: int, device="cpu") -> torch.Tensor:
        """Raw queries of question k's own tokens at one layer: [n_k, Hq, D]."""
        g = self.geom
        n = int(self.q_len[k])
        return self._gen(Q_QST, k, (n, g.n_q_heads, g.head_dim), layer * n, device)

    def _step_rows(self, kind: int, s: int, layer: int, qids, heads: int, device) -> torch.Tensor:
        g = self.geom
        NQ = self.n_questions
        qids = torch.as_tensor(np.asarray(qids), dtype=torch.int64, device=device)
        inner = heads * g.head_dim
        base = (layer * NQ + qids) * inner
        idx = base[:, None] + torch.arange(inner, dtype=torch.int64, device=device)[None, :]
        return values_at(self.seed, stream_id(kind, s), idx).view(len(qids), heads, g.head_dim)

    def step_q(self, s: int, layer: int, qids, device="cpu") -> torch.Tensor:
        """Raw queries fed at decode step s for the given global question ids: [len, Hq, D]."""
        return self._step_rows(Q_STEP, s, layer, qids, self.geom.n_q_heads, device)

    def step_kv(self, s: int, layer: int, qids, device="cpu"):
        """Raw K and V of the answer token fed at step s (y_{s+1}) for the given questions."""
        h = self.geom.n_kv_heads
        return (self._step_rows(K_STEP, s, layer, qids, h, device),
                self._step_rows(V_STEP, s, layer, qids, h, device))


LLAMA3_8B = Geometry(32, 32, 8, 128, 5e5)
LLAMA3_70B = Geometry(80, 64, 8, 128, 5e5)
SMALL = Geometry(1, 8, 2, 64, 1e4)

_BASE_SEED = 260905707000


def make_workload(name: str, n_layers: Optional[int] = None) -> Workload:
    """The five benchmark configurations (all ranges inclusive).

    C1 small parity case; C2 Llama-3-8B geometry, one prompt; C3 long context with
    per-question stop steps; C4 batched ragged prompts; C5 many questions, 70B geometry.
    `n_layers` overrides the layer count (tests use fewer layers; values of the
    layers kept are unchanged because the layer is the slowest index only within
    a layer's own slice for per-token tensors -- see ctx_kv/question_kv).
    """
    if name.startswith("SWEEP-"):
        return _sweep_workload(name, n_layers)
    if name.startswith("S"):
        return _shape_workload(name, n_layers)
    c = int(name[1:])
    seed = _BASE_SEED + c
    ri = lambda tag, i, lo, hi: _randint(seed, tag, i, lo, hi)
    if c == 1:
        geom, B, n_steps = SMALL, 1, 32
        ctx = [512]; qc = [4]; ql = (8, 24); stop_rng = None
    elif c == 2:
        geom, B, n_steps = LLAMA3_8B, 1, 128
        ctx = [2048]; qc = [16]; ql = (16, 48); stop_rng = None
    elif c == 3:
        geom, B, n_steps = LLAMA3_8B, 1, 256
        ctx = [16384]; qc = [32]; ql = (16, 64); stop_rng = (8, 256)
    elif c == 4:
        geom, B, n_steps = LLAMA3_8B, 32, 128
        ctx = [ri(1, b, 1024, 4096) for b in range(B)]
        qc = [ri(2, b, 4, 64) for b in range(B)]
        ql = (8, 48); stop_rng = None
    elif c == 5:
        geom, B, n_steps = LLAMA3_70B, 4, 64
        ctx = [8192] * 4; qc = [256] * 4; ql = (8, 32); stop_rng = (1, 64)
    else:
        raise ValueError(name)
    if n_layers is not None:
        geom = Geometry(n_layers, geom.n_q_heads, geom.n_kv_heads, geom.head_dim, geom.rope_theta)
    NQ = sum(qc)
    q_len = np.array([ri(3, k, ql[0], ql[1]) for k in range(NQ)], dtype=np.int32)
    if stop_rng is None:
        stop = np.full(NQ, n_steps, dtype=np.int32)
    else:
        stop = np.array([ri(4, k, stop_rng[0], stop_rng[1]) for k in range(NQ)], dtype=np.int32)
        n_steps = int(stop.max())
    return Workload(name, geom, seed, np.array(ctx, dtype=np.int32), np.array(qc, dtype=np.int32),
                    q_len, stop, stop.copy(), n_steps)


def _shape_workload(name: str, n_layers: Optional[int] = None) -> Workload:
    """A second family of synthetic shapes, sized like the rows of the paper's dataset table (context + instruction
    length, questions per context, question length, answer length; Sec. 5, Table "dataset info") with six stacked
    prompts per batch, Llama-3-8B attention geometry.  All ranges inclusive, drawn per prompt / per question:

    S1  long contexts, many questions, short answers: L ~ U{2600..4400}, Q ~ U{22..38}, n ~ U{8..16}, stop ~ U{6..40}
    S2  short contexts, few questions:                L ~ U{170..280},   Q ~ U{6..12},  n ~ U{9..17}, stop ~ U{4..30}
    S3  a long instruction shared by the whole batch (few-shot examples, kept once): P = 2754 tokens, twelve prompts
        (three stacked prompts of four contexts in the paper's terms) with L ~ U{550..920}, Q ~ U{22..38},
        n ~ U{8..16}, stop ~ U{1..11}
    """
    c = int(name[1:])
    seed = _BASE_SEED + 100 + c
    ri = lambda tag, i, lo, hi: _randint(seed, tag, i, lo, hi)
    B, shared = 6, 0
    if c == 1:
        Lr, Qr, nr, sr = (2600, 4400), (22, 38), (8, 16), (6, 40)
    elif c == 3:
        B, shared = 12, 2754
        Lr, Qr, nr, sr = (550, 920), (22, 38), (8, 16), (1, 11)
    elif c == 2:
        Lr, Qr, nr, sr = (170, 280), (6, 12), (9, 17), (4, 30)
    else:
        raise ValueError(name)
    geom = LLAMA3_8B
    if n_layers is not None:
        geom = Geometry(n_layers, geom.n_q_heads, geom.n_kv_heads, geom.head_dim, geom.rope_theta)
    ctx = [ri(1, b, *Lr) for b in range(B)]
    qc = [ri(2, b, *Qr) for b in range(B)]
    NQ = sum(qc)
    q_len = np.array([ri(3, k, *nr) for k in range(NQ)], dtype=np.int32)
    stop = np.array([ri(4, k, *sr) for k in range(NQ)], dtype=np.int32)
    return Workload(name, geom, seed, np.array(ctx, dtype=np.int32), np.array(qc, dtype=np.int32), q_len, stop,
                    stop.copy(), int(stop.max()), shared)


SWEEP_CONTEXTS = (2048, 4096, 8192, 16384)
SWEEP_QUESTIONS = (1, 2, 4, 8, 16, 32)


def _sweep_workload(name: str, n_layers: Optional[int] = None) -> Workload:
    """The axes of the paper's ablations (App. C: questions per context 1..32, context length 1x..8x) as named
    workloads "SWEEP-L<context>-Q<questions>": one prompt with a context of L tokens and Q questions of 32 tokens each,
    16 decode steps without stop steps, Llama-3-8B geometry."""
    parts = name.split("-")
    L, Q = int(parts[1][1:]), int(parts[2][1:])
    assert parts[0] == "SWEEP" and 1 <= L <= (1 << 20) and 1 <= Q <= 4096, name
    geom = LLAMA3_8B
    if n_layers is not None:
        geom = Geometry(n_layers, geom.n_q_heads, geom.n_kv_heads, geom.head_dim, geom.rope_theta)
    seed = _BASE_SEED + 1000 + 64 * (L // 1024) + Q
    stop = np.full(Q, 16, dtype=np.int32)
    return Workload(name, geom, seed, np.array([L], dtype=np.int32), np.array([Q], dtype=np.int32),
                    np.full(Q, 32, dtype=np.int32), stop, stop.copy(), 16)


def custom_workload(name: str, geom: Geometry, seed: int, ctx_len: List[int], q_count: List[int],
                    q_len: List[int], stop: List[int], max_new: Optional[List[int]] = None,
                    shared_len: int = 0) -> Workload:
    stop_a = np.array(stop, dtype=np.int32)
    mn = stop_a.copy() if max_new is None else np.array(max_new, dtype=np.int32)
    return Workload(name, geom, seed, np.array(ctx_len, dtype=np.int32), np.array(q_count, dtype=np.int32),
                    np.array(q_len, dtype=np.int32), stop_a, mn, int(stop_a.max()), shared_len)
