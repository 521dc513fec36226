"""CPU fp64 oracle for the IPPD decode-attention path.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this
module; the product (the CUDA library and its Python binding) never does, and it
shares no code, table or helper with the CUDA path.  Inputs are plain numpy
arrays handed in by the caller.

What is defined here (paper sections in brackets):

* `standalone_attend`  -- the result itself: the attention output of one
  question prompted ALONE as (context, question, answer-so-far) with ordinary
  position ids 0..T-1 and a causal last row [Sec. 3 problem formulation; Sec. 4.2:
  the IPPD output of an answer token equals this].  Pinned by: the library SDPA on
  the Q=1 case, closed-form softmax cases, RoPE closed forms / complex-number form.
* `rope`               -- rotary embedding, rotate-half pairing (i, i+D/2),
  angle pos * theta^(-2i/D) (the position-id convention of the HF models the
  paper runs; the paper itself only speaks of position ids).
* `layout`             -- virtual position ids, context / question ids of the
  stacked header, branch offsets [Sec. 4.1 virtual-position equations; App. A.1].
* `stacked_sequence`, `dense_mask`, `dense_attend` -- the paper's own dense
  formulation: the stacked token sequence, the three mask predicates and
  softmax(QK^T/sqrt(d) + M)V over it [Sec. 4.1 mask equations, Sec. 4.2].  Used on
  tiny inputs to show that it agrees with `standalone_attend` (the paper's
  equivalence claim) and that the structural attended set equals the predicates.

* `standalone_prefill`, `prefill_tuple` -- the prefill of the stacked header: every header row
  equals the row of its own standalone causal prompt [Sec. 4, Sec. 4.2].  Pinned by: the library
  SDPA with is_causal, and the dense formulation (header rows under the dense mask).
* `tuple_inputs`, `attend_tuple` -- assemble the standalone prompt of one (prompt,
  question, step, layer, KV head) from a workload's raw accessors and evaluate it.
  Pinned by: the dense formulation over a stacked sequence assembled independently
  in the tests, with the KV head of each query head chosen by an explicit repeat.

* `quantize_e4m3`      -- the 8-bit cache variant (not in the paper: a storage format of this build): the
  rotated key and the value are kept as e4m3 numbers (1 sign, 4 exponent bits with bias 7, 3 mantissa bits,
  subnormals, largest magnitude 448, no infinity), rounded to nearest-even and saturating; `standalone_attend(...,
  kv_e4m3=True)` and `attend_tuple(..., kv_e4m3=True)` evaluate the same definition over the quantised keys and
  values.  Pinned by: the enumeration of all 254 finite codes, hand values, and the library's float8 cast.

Numeric attention values: parity unpinned by the paper (it prints no attention
value); every function here is pinned by the library routine, closed forms and
invariants named above, in tests/test_oracle_pins.py.
"""
from __future__ import annotations

import numpy as np

INT32_MAX = 2**31 - 1


# --------------------------------------------------------------------------- floats
def rope(x: np.ndarray, pos, theta: float) -> np.ndarray:
    """Rotate x[..., D] to position `pos` (broadcast over leading dims), in fp64."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    i = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / D)
    phi = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(phi), np.sin(phi)
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def quantize_e4m3(x: np.ndarray) -> np.ndarray:
    """Nearest e4m3 number (ties to even mantissa, magnitudes beyond 448 saturate to 448), returned as fp64.

    e4m3: value = (-1)^s * 2^(e-7) * (1 + m/8) for exponent field e in 1..15 and mantissa m in 0..7 (e = 15, m = 7 is
    not a number and never produced), and (-1)^s * 2^-6 * m/8 for e = 0.  So the numbers are spaced 2^(E-3) apart in
    the binade [2^E, 2^(E+1)), E >= -6, and 2^-9 apart below 2^-6.
    """
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    E = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))  # binade of |x|; everything below 2^-6 uses the subnormal spacing
    step = 2.0 ** (E - 3)
    q = np.rint(a / step) * step  # np.rint rounds halves to even
    return np.sign(x) * np.minimum(q, 448.0)


def standalone_attend(k_raw: np.ndarray, v_raw: np.ndarray, q_raw: np.ndarray, theta: float,
                      kv_e4m3: bool = False) -> np.ndarray:
    """Attention output of the LAST token of one standalone prompt.

    k_raw, v_raw: [T, D] raw keys / values of the prompt's T tokens (context tokens,
    then question tokens, then the answer tokens fed so far, the last one being the
    token whose query is evaluated).  q_raw: [H, D] raw queries of that last token
    for the H query heads that share this KV head.  Ordinary positions 0..T-1; the
    query sits at T-1 and sees all T keys (itself included).  Returns [H, D] fp64.
    kv_e4m3: the rotated keys and the values are the e4m3 numbers nearest to them (the 8-bit cache variant).
    """
    k_raw = np.asarray(k_raw, dtype=np.float64)
    v = np.asarray(v_raw, dtype=np.float64)
    q_raw = np.asarray(q_raw, dtype=np.float64)
    T, D = k_raw.shape
    k = rope(k_raw, np.arange(T), theta)
    if kv_e4m3:
        k, v = quantize_e4m3(k), quantize_e4m3(v)
    q = rope(q_raw, np.full(q_raw.shape[0], T - 1), theta)
    z = (q @ k.T) / np.sqrt(D)
    z = z - z.max(axis=-1, keepdims=True)
    p = np.exp(z)
    p = p / p.sum(axis=-1, keepdims=True)
    return p @ v


def standalone_prefill(k_raw: np.ndarray, v_raw: np.ndarray, q_raw: np.ndarray, theta: float,
                       kv_e4m3: bool = False) -> np.ndarray:
    """Causal self-attention of ONE standalone prompt, every row (the prefill of a triplet prompted alone).

    k_raw, v_raw: [T, D] raw keys / values of the prompt's T tokens; q_raw: [T, H, D] raw queries of the same tokens
    for the H query heads that share this KV head.  Ordinary positions 0..T-1; row i sees keys 0..i.  Returns
    [T, H, D] fp64.  [Sec. 4: the stacked header is prefilled once; Sec. 4.2: every token of the stacked prompt follows
    the computation of its own standalone prompt.]
    """
    k_raw = np.asarray(k_raw, dtype=np.float64)
    v = np.asarray(v_raw, dtype=np.float64)
    q_raw = np.asarray(q_raw, dtype=np.float64)
    T, D = k_raw.shape
    pos = np.arange(T)
    k = rope(k_raw, pos, theta)
    if kv_e4m3:  # the 8-bit cache variant: every row reads the stored numbers, its own token's included
        k, v = quantize_e4m3(k), quantize_e4m3(v)
    out = np.empty_like(q_raw)
    causal = np.tril(np.ones((T, T), dtype=bool))
    for h in range(q_raw.shape[1]):
        q = rope(q_raw[:, h], pos, theta)
        z = (q @ k.T) / np.sqrt(D)
        z = np.where(causal, z, -np.inf)
        z = z - z.max(axis=-1, keepdims=True)
        p = np.exp(z)
        p = p / p.sum(axis=-1, keepdims=True)
        out[:, h] = p @ v
    return out


# --------------------------------------------------------------------------- integers
def layout(ctx_len, q_count, q_len, max_new, branch_align: int, tile_tokens: int, shared_len: int = 0) -> dict:
    """Integer tables of a batch of stacked prompts (one context per prompt, an optional
    instruction of `shared_len` tokens shared by all prompts).

    Header = the shared instruction's tokens (context id 0, question id 0), then per
    prompt b its context tokens and its questions' tokens in order.  With P = shared_len,
    virtual positions: instruction token i -> i; context token i -> P + i; token j of
    question k -> P + L_b + j; the answer token fed at decode step s -> P + L_b + n_k + s
    [Sec. 4.1].  Context ids are 1-based per prompt, question ids are global and
    1-based, 0 marks shared tokens.  The instruction owns the first ceil(P / tile_tokens)
    tiles.  Branch k owns slots
    [branch_off[k], branch_off[k+1]) with capacity n_k + max_new_k rounded up to
    `branch_align`; the answer token of step s lives at slot branch_off[k]+n_k+s.
    Context b owns tiles [ctx_tile_off[b], ctx_tile_off[b+1]) of `tile_tokens` tokens.
    """
    B = len(ctx_len)
    q_begin = [0]
    for b in range(B):
        q_begin.append(q_begin[-1] + int(q_count[b]))
    NQ = q_begin[-1]
    P = int(shared_len)
    prompt_of, branch_off, hdr_begin = [], [0], [P]
    pos, cid, qid = [], [], []
    for i in range(P):
        pos.append(i); cid.append(0); qid.append(0)
    ctx_tile_off = [(P + tile_tokens - 1) // tile_tokens]
    for b in range(B):
        L = int(ctx_len[b])
        ctx_tile_off.append(ctx_tile_off[-1] + (L + tile_tokens - 1) // tile_tokens)
        for i in range(L):
            pos.append(P + i); cid.append(b + 1); qid.append(0)
        for k in range(q_begin[b], q_begin[b + 1]):
            prompt_of.append(b)
            for j in range(int(q_len[k])):
                pos.append(P + L + j); cid.append(b + 1); qid.append(k + 1)
            cap = int(q_len[k]) + int(max_new[k])
            cap = (cap + branch_align - 1) // branch_align * branch_align
            branch_off.append(branch_off[-1] + cap)
        hdr_begin.append(len(pos))
    i32 = lambda a: np.asarray(a, dtype=np.int32)
    return {
        "q_begin": i32(q_begin), "prompt_of": i32(prompt_of), "branch_off": np.asarray(branch_off, dtype=np.int64),
        "hdr_begin": np.asarray(hdr_begin, dtype=np.int64), "hdr_pos_virt": i32(pos), "hdr_ctx_id": i32(cid),
        "hdr_qtn_id": i32(qid), "ctx_tile_off": i32(ctx_tile_off), "n_questions": NQ,
    }


def step_position(ctx_len_b: int, q_len_k: int, s: int, shared_len: int = 0) -> int:
    """Virtual position of the answer token fed at decode step s (the paper's t = s+1)."""
    return shared_len + ctx_len_b + q_len_k + s


def stacked_sequence(p_len: int, ctx_lens, q_lens, n_answer, n_pad: int = 0):
    """(pos_virt, ctx, qtn) of every token of ONE stacked prompt in physical order.

    p_len: length of the shared instruction p (ctx = qtn = 0).  ctx_lens[j]: length
    of context j (1-based id j+1).  q_lens[j][k]: question lengths under context j.
    n_answer[j][k]: answer tokens appended so far for that question.  Order: header
    [p, c_1, x_11, x_12, .., c_2, ..], then the answer tokens in generation order
    (step-major: all t=1 tokens in question order, then t=2, ..), then `n_pad` pad
    tokens with position INT32_MAX and ids -1 (batching rule of Sec. 4.4).
    Also returns, per token, a tag (kind, j, k, t) to find rows in tests.
    """
    pos, ctx, qtn, tag = [], [], [], []
    for i in range(p_len):
        pos.append(i); ctx.append(0); qtn.append(0); tag.append(("p", 0, 0, i))
    gq = 0
    qid_of = {}
    for j, Lc in enumerate(ctx_lens):
        for i in range(Lc):
            pos.append(p_len + i); ctx.append(j + 1); qtn.append(0); tag.append(("c", j, 0, i))
        for k, n in enumerate(q_lens[j]):
            gq += 1
            qid_of[(j, k)] = gq
            for i in range(n):
                pos.append(p_len + Lc + i); ctx.append(j + 1); qtn.append(gq); tag.append(("x", j, k, i))
    max_t = max([0] + [a for row in n_answer for a in row])
    for t in range(max_t):
        for j, Lc in enumerate(ctx_lens):
            for k, n in enumerate(q_lens[j]):
                if n_answer[j][k] > t:
                    pos.append(p_len + Lc + n + t); ctx.append(j + 1); qtn.append(qid_of[(j, k)])
                    tag.append(("y", j, k, t))
    for i in range(n_pad):
        pos.append(INT32_MAX); ctx.append(-1); qtn.append(-1); tag.append(("pad", 0, 0, i))
    return np.asarray(pos, dtype=np.int64), np.asarray(ctx, dtype=np.int64), np.asarray(qtn, dtype=np.int64), tag


def dense_mask(pos, ctx, qtn) -> np.ndarray:
    """M_fin[q, k] = M_caus and M_ctx and M_qtn, evaluated for every pair (bool [n, n])."""
    n = len(pos)
    m = np.zeros((n, n), dtype=bool)
    for q in range(n):
        for k in range(n):
            caus = pos[q] >= pos[k]
            mctx = (ctx[q] == ctx[k]) or (ctx[k] == 0)
            mqtn = (qtn[q] == qtn[k]) or (qtn[k] == 0)
            m[q, k] = caus and mctx and mqtn
    return m


def dense_attend(q_raw, k_raw, v_raw, pos, mask, theta: float) -> np.ndarray:
    """softmax(Q K^T / sqrt(D) + M) V over a stacked sequence, RoPE at the virtual positions.

    q_raw, k_raw, v_raw: [n, D] (one head).  mask: bool [n, n], True = attend
    (additive 0), False = -inf.  Rows with no attended key return NaN.
    """
    q = rope(q_raw, pos, theta)
    k = rope(k_raw, pos, theta)
    v = np.asarray(v_raw, dtype=np.float64)
    D = q.shape[-1]
    z = (q @ k.T) / np.sqrt(D)
    z = np.where(mask, z, -np.inf)
    with np.errstate(invalid="ignore"):
        z = z - z.max(axis=-1, keepdims=True)
        p = np.exp(z)
        p = p / p.sum(axis=-1, keepdims=True)
    return p @ v


# --------------------------------------------------------------------------- per-tuple driver
def tuple_inputs(wl, b: int, k: int, s: int, layer: int, kv_head: int, ctx_cache: dict | None = None,
                 step_cache: dict | None = None):
    """Raw tensors of the standalone prompt of question k (global id) of prompt b at decode step s, one layer, one KV
    head: (k_raw [T, D], v_raw [T, D], q_raw [G, D]) in fp64, T = P + L_b + n_k + s + 1.

    The prompt is the instruction shared by the batch (P = wl.shared_len tokens, if the workload has one), the
    context tokens, the question's tokens, then the answer tokens fed at steps 0..s (the last one is
    the token whose query is evaluated; Sec. 3, Sec. 4.2).  The G query heads [kv_head*G, (kv_head+1)*G) share KV head
    `kv_head`.  `wl` is any object with the raw-tensor accessors of a workload (ctx_kv, question_kv, step_kv, step_q,
    geom); the caches only avoid regenerating the same raw tensors.
    """
    g = wl.geom
    G = g.n_q_heads // g.n_kv_heads
    key = (b, layer, kv_head)
    if ctx_cache is not None and key in ctx_cache:
        kc, vc = ctx_cache[key]
    else:
        kc, vc = wl.ctx_kv(b, layer)
        kc = kc[:, kv_head].double().numpy()
        vc = vc[:, kv_head].double().numpy()
        if ctx_cache is not None:
            ctx_cache[key] = (kc, vc)
    kq, vq = wl.question_kv(k, layer)
    ks = [kc, kq[:, kv_head].double().numpy()]
    vs = [vc, vq[:, kv_head].double().numpy()]
    if getattr(wl, "shared_len", 0) > 0:  # the triplet's prompt starts with the instruction p (Sec. 3: (p, c_j, x_jk))
        skey = ("shared", layer, kv_head)
        if ctx_cache is not None and skey in ctx_cache:
            kp, vp = ctx_cache[skey]
        else:
            kp, vp = wl.shared_kv(layer)
            kp, vp = kp[:, kv_head].double().numpy(), vp[:, kv_head].double().numpy()
            if ctx_cache is not None:
                ctx_cache[skey] = (kp, vp)
        ks.insert(0, kp)
        vs.insert(0, vp)
    if step_cache is None:
        for t in range(s + 1):
            ka, va = wl.step_kv(t, layer, [k])
            ks.append(ka[0][None, kv_head].double().numpy())
            vs.append(va[0][None, kv_head].double().numpy())
    else:
        # raw step tensors of ALL questions for one (layer, KV head), generated once per step and kept stacked over the
        # steps, [steps so far, NQ, D]: a question's answer tokens are then one slice
        key = ("steps", layer, kv_head)
        kst, vst = step_cache.get(key, (np.zeros((0, wl.n_questions, g.head_dim)),) * 2)
        if kst.shape[0] < s + 1:
            more = [wl.step_kv(t, layer, list(range(wl.n_questions))) for t in range(kst.shape[0], s + 1)]
            kst = np.concatenate([kst] + [a[:, kv_head].double().numpy()[None] for a, _ in more])
            vst = np.concatenate([vst] + [b_[:, kv_head].double().numpy()[None] for _, b_ in more])
            step_cache[key] = (kst, vst)
        ks.append(kst[:s + 1, k])
        vs.append(vst[:s + 1, k])
    q = wl.step_q(s, layer, [k])[0, kv_head * G:(kv_head + 1) * G].double().numpy()
    return np.concatenate(ks), np.concatenate(vs), q


def attend_tuple(wl, b: int, k: int, s: int, layer: int, kv_head: int, ctx_cache: dict | None = None,
                 step_cache: dict | None = None, kv_e4m3: bool = False) -> np.ndarray:
    """Oracle output for question k (global id) of prompt b at decode step s, one layer, all query heads of one KV
    head: [G, D] fp64 -- `standalone_attend` on the standalone prompt assembled by `tuple_inputs`.  Pinned by the
    dense-mask formulation assembled independently in the tests (the equivalence of Sec. 4.2)."""
    k_raw, v_raw, q_raw = tuple_inputs(wl, b, k, s, layer, kv_head, ctx_cache, step_cache)
    return standalone_attend(k_raw, v_raw, q_raw, wl.geom.rope_theta, kv_e4m3)


def prefill_tuple(wl, b: int, k: int | None, layer: int, kv_head: int, kv_e4m3: bool = False) -> np.ndarray:
    """Oracle prefill outputs of the header rows of one standalone prompt, one layer, all query heads of one KV head.

    k = a global question id: the prompt is (instruction p, context c_b, question x_k); returns the rows of the
    question's tokens, [n_k, G, D].  k = None: the prompt is (p, c_b) alone; returns the rows of p and c_b,
    [P + L_b, G, D] (a context row does not depend on the questions behind it).  Uses the workload's header query
    accessors (shared_q, ctx_q, question_q) next to the key/value accessors.
    """
    g = wl.geom
    G = g.n_q_heads // g.n_kv_heads
    hs = slice(kv_head * G, (kv_head + 1) * G)
    ks, vs, qs = [], [], []
    if getattr(wl, "shared_len", 0) > 0:
        kp, vp = wl.shared_kv(layer)
        ks.append(kp[:, kv_head]); vs.append(vp[:, kv_head]); qs.append(wl.shared_q(layer)[:, hs])
    kc, vc = wl.ctx_kv(b, layer)
    ks.append(kc[:, kv_head]); vs.append(vc[:, kv_head]); qs.append(wl.ctx_q(b, layer)[:, hs])
    if k is not None:
        kq, vq = wl.question_kv(k, layer)
        ks.append(kq[:, kv_head]); vs.append(vq[:, kv_head]); qs.append(wl.question_q(k, layer)[:, hs])
    cat = lambda ts: np.concatenate([t.double().numpy() for t in ts])
    out = standalone_prefill(cat(ks), cat(vs), cat(qs), g.rope_theta, kv_e4m3)
    return out if k is None else out[-int(wl.q_len[k]):]
