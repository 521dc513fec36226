"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test names the fact that fixes the value: a textbook closed form, a library
routine, an invariant the paper states, or brute force on a tiny input.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ippd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ RoPE
def _parse_pos(tok):
    return {"pi": math.pi, "2pi": 2 * math.pi, "0": 0.0}[tok]


def test_rope_special_angles_golden():
    # closed forms at angles pi/2, pi, 2*pi (fixture explains each line)
    rows = [l.split() for l in open(os.path.join(GOLDEN, "rope_special_angles.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        pos = _parse_pos(r[0])
        x = np.array([float(v) for v in r[1:5]])
        want = np.array([float(v) for v in r[5:9]])
        got = orc.rope(x[None, :], np.array([pos]), 4.0)[0]
        np.testing.assert_allclose(got, want, atol=1e-14)


def test_rope_equals_complex_rotation():
    # rotate-half RoPE is multiplication of z_i = x_i + 1j*x_{i+D/2} by exp(1j*pos*theta^(-2i/D))
    D, theta = 16, 1e4
    x = rng.standard_normal((7, D))
    pos = np.array([0, 1, 2, 17, 300, 4095, 16383])
    z = x[:, : D // 2] + 1j * x[:, D // 2:]
    w = np.exp(1j * pos[:, None] * theta ** (-np.arange(D // 2) / (D / 2)))
    zz = z * w
    want = np.concatenate([zz.real, zz.imag], axis=-1)
    np.testing.assert_allclose(orc.rope(x, pos, theta), want, atol=1e-12)


def test_rope_norm_identity_and_relative_property():
    D, theta = 64, 5e5
    x = rng.standard_normal((5, D))
    y = rng.standard_normal((5, D))
    np.testing.assert_array_equal(orc.rope(x, np.zeros(5), theta), x)
    np.testing.assert_allclose(np.linalg.norm(orc.rope(x, np.arange(5) * 1000, theta), axis=-1),
                               np.linalg.norm(x, axis=-1), rtol=1e-13)
    # the score of (q at m, k at n) depends on m - n only
    m, n, shift = 900, 37, 5000
    a = (orc.rope(x, np.full(5, m), theta) * orc.rope(y, np.full(5, n), theta)).sum(-1)
    b = (orc.rope(x, np.full(5, m + shift), theta) * orc.rope(y, np.full(5, n + shift), theta)).sum(-1)
    np.testing.assert_allclose(a, b, atol=1e-9)
    # and it is NOT symmetric in (m, n): catches a sign error in the rotation
    c = (orc.rope(x, np.full(5, n), theta) * orc.rope(y, np.full(5, m), theta)).sum(-1)
    assert np.abs(a - c).max() > 1e-3


# ------------------------------------------------------------------ attention: closed forms
def test_attend_zero_query_is_mean_of_values():
    T, D = 37, 8
    k = rng.standard_normal((T, D)); v = rng.integers(-4, 5, (T, D)).astype(float)
    out = orc.standalone_attend(k, v, np.zeros((3, D)), 1e4)
    np.testing.assert_allclose(out, np.broadcast_to(v.mean(0), (3, D)), atol=1e-13)


def test_attend_constant_values_and_dominant_key():
    T, D = 50, 16
    k = rng.standard_normal((T, D)); q = rng.standard_normal((2, D))
    c = rng.standard_normal(D)
    np.testing.assert_allclose(orc.standalone_attend(k, np.tile(c, (T, 1)), q, 1e4), np.tile(c, (2, 1)), atol=1e-13)
    # last key = 200*q (same position as the query, so RoPE cancels): softmax is one-hot on it
    v = rng.standard_normal((T, D))
    k2 = k.copy(); k2[-1] = 200.0 * q[0]
    np.testing.assert_allclose(orc.standalone_attend(k2, v, q[:1], 1e4)[0], v[-1], atol=1e-12)


def test_attend_two_keys_three_to_one():
    # key 0 is the zero vector (score 0); key 1 = c*q sits at the query's own position, so its
    # score is c*|q|^2/sqrt(D) = ln 3: the weights are exactly 1/4 and 3/4 (checks scale, exp, norm)
    D = 8
    q = rng.standard_normal((1, D))
    c = math.log(3.0) * math.sqrt(D) / float((q ** 2).sum())
    k = np.stack([np.zeros(D), c * q[0]])
    v = rng.standard_normal((2, D))
    out = orc.standalone_attend(k, v, q, 5e5)[0]
    np.testing.assert_allclose(out, 0.25 * v[0] + 0.75 * v[1], atol=1e-13)


def test_attend_matches_library_sdpa_last_row():
    # Q=1 is ordinary causal decode: compare with torch's scaled_dot_product_attention (fp64),
    # feeding it keys/queries rotated by the complex-number form of RoPE (not by oracle.rope)
    T, D, H, theta = 83, 32, 4, 1e4
    k = rng.standard_normal((T, D)); v = rng.standard_normal((T, D)); qfull = rng.standard_normal((H, T, D))

    def crope(x, pos):
        z = x[..., : D // 2] + 1j * x[..., D // 2:]
        w = np.exp(1j * np.asarray(pos)[..., None] * theta ** (-2.0 * np.arange(D // 2) / D))
        zz = z * w
        return np.concatenate([zz.real, zz.imag], -1)

    kt = torch.from_numpy(crope(k, np.arange(T)))[None, None].expand(1, H, T, D)
    vt = torch.from_numpy(v)[None, None].expand(1, H, T, D)
    qt = torch.from_numpy(crope(qfull, np.arange(T)[None, :]))[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)[0, :, -1].numpy()
    got = orc.standalone_attend(k, v, qfull[:, -1], theta)
    np.testing.assert_allclose(got, ref, atol=1e-12)


# ------------------------------------------------------------------ masks
def test_mask_fig2_golden():
    want = np.array([[int(t) for t in l.split()] for l in open(os.path.join(GOLDEN, "fig2_mask.txt"))
                     if l.strip() and l[0] != "#"], dtype=bool)
    pos, ctx, qtn, tag = orc.stacked_sequence(1, [1, 1], [[1, 1], [1, 1]], [[1, 1], [1, 1]])
    assert [t[0] + (str(t[1] + 1) if t[0] != "p" else "") for t in tag] == \
        ["p", "c1", "x1", "x1", "c2", "x2", "x2", "y1", "y1", "y2", "y2"]
    np.testing.assert_array_equal(orc.dense_mask(pos, ctx, qtn), want)


def _structural_rows(p_len, ctx_lens, q_lens, n_answer, tag):
    """Attended set written as 'p + own context + own question/answer prefix up to self'."""
    n = len(tag)
    m = np.zeros((n, n), dtype=bool)
    for r, (kind, j, k, i) in enumerate(tag):
        for c, (kind2, j2, k2, i2) in enumerate(tag):
            if kind == "pad" or kind2 == "pad":
                continue
            if kind2 == "p":
                ok = kind != "p" or i2 <= i
            elif kind2 == "c":
                ok = kind != "p" and j2 == j and (kind != "c" or i2 <= i)
            elif kind2 == "x":
                ok = kind in ("x", "y") and (j2, k2) == (j, k) and (kind == "y" or i2 <= i)
            else:  # answer key
                ok = kind == "y" and (j2, k2) == (j, k) and i2 <= i
            m[r, c] = ok
    return m


@pytest.mark.parametrize("case", [
    (2, [3], [[2, 4, 1]], [[3, 0, 2]], 0),
    (0, [5], [[3, 3]], [[1, 1]], 2),
    (1, [2, 4, 3], [[1], [2, 2, 3, 1], [2, 2]], [[2], [0, 1, 3, 2], [1, 1]], 1),
])
def test_mask_predicates_equal_structural_set(case):
    p_len, ctx_lens, q_lens, n_answer, n_pad = case
    pos, ctx, qtn, tag = orc.stacked_sequence(p_len, ctx_lens, q_lens, n_answer, n_pad)
    m = orc.dense_mask(pos, ctx, qtn)
    rows = [r for r, t in enumerate(tag) if t[0] != "pad"]
    np.testing.assert_array_equal(m[rows], _structural_rows(p_len, ctx_lens, q_lens, n_answer, tag)[rows])
    # nobody attends to a pad column (position INT_MAX), Sec. 4.4
    pads = [c for c, t in enumerate(tag) if t[0] == "pad"]
    assert not m[np.ix_(rows, pads)].any()
    # row of answer token (j,k,t) has exactly |p| + |c_j| + |x_jk| + t + 1 attended keys
    for r, (kind, j, k, t) in enumerate(tag):
        if kind == "y":
            assert m[r].sum() == p_len + ctx_lens[j] + q_lens[j][k] + t + 1
            assert pos[r] == p_len + ctx_lens[j] + q_lens[j][k] + t  # virtual-position equation, Sec. 4.1


# ------------------------------------------------------------------ the paper's equivalence claim
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_dense_masked_attention_equals_standalone_prompts(seed):
    r = np.random.default_rng(seed)
    D, theta = 8, 1e4
    p_len = int(r.integers(0, 3))
    ctx_lens = [int(v) for v in r.integers(1, 6, size=r.integers(1, 4))]
    q_lens = [[int(v) for v in r.integers(1, 4, size=r.integers(1, 4))] for _ in ctx_lens]
    n_answer = [[int(v) for v in r.integers(0, 4, size=len(q))] for q in q_lens]
    pos, ctx, qtn, tag = orc.stacked_sequence(p_len, ctx_lens, q_lens, n_answer)
    n = len(pos)
    q_raw, k_raw, v_raw = r.standard_normal((3, n, D))
    dense = orc.dense_attend(q_raw, k_raw, v_raw, pos, orc.dense_mask(pos, ctx, qtn), theta)
    checked = 0
    for row, (kind, j, k, t) in enumerate(tag):
        if kind != "y":
            continue
        # the standalone prompt of this triplet: p, c_j, x_jk, y_1..y_{t+1}, in that order
        idx = [c for c, (k2, j2, kk2, t2) in enumerate(tag)
               if k2 == "p" or (k2 == "c" and j2 == j) or (k2 == "x" and (j2, kk2) == (j, k))
               or (k2 == "y" and (j2, kk2) == (j, k) and t2 <= t)]
        alone = orc.standalone_attend(k_raw[idx], v_raw[idx], q_raw[row][None], theta)[0]
        np.testing.assert_allclose(dense[row], alone, atol=1e-12)
        checked += 1
    assert checked == sum(sum(a) for a in n_answer)


# ------------------------------------------------------------------ layout
def test_layout_positions_are_standalone_positions():
    ctx_len = [5, 0, 130]; q_count = [2, 1, 3]
    q_len = [3, 1, 4, 2, 9, 1]; max_new = [4, 1, 130, 7, 1, 2]
    lay = orc.layout(ctx_len, q_count, q_len, max_new, branch_align=8, tile_tokens=128)
    np.testing.assert_array_equal(lay["q_begin"], [0, 2, 3, 6])
    np.testing.assert_array_equal(lay["prompt_of"], [0, 0, 1, 2, 2, 2])
    np.testing.assert_array_equal(lay["ctx_tile_off"], [0, 1, 1, 3])
    # capacities: round_up(n+max_new, 8) = 8, 8, 136, 16, 16, 8
    np.testing.assert_array_equal(lay["branch_off"], [0, 8, 16, 152, 168, 184, 192])
    # brute force: walk each standalone triplet and record the ordinary position of every header token
    h = 0
    for b in range(3):
        assert lay["hdr_begin"][b] == h
        for i in range(ctx_len[b]):
            assert (lay["hdr_pos_virt"][h], lay["hdr_ctx_id"][h], lay["hdr_qtn_id"][h]) == (i, b + 1, 0); h += 1
        for k in range(lay["q_begin"][b], lay["q_begin"][b + 1]):
            standalone = list(range(ctx_len[b] + q_len[k]))  # positions of (context, question) alone
            for j in range(q_len[k]):
                assert lay["hdr_pos_virt"][h] == standalone[ctx_len[b] + j]
                assert (lay["hdr_ctx_id"][h], lay["hdr_qtn_id"][h]) == (b + 1, k + 1); h += 1
    assert lay["hdr_begin"][3] == h == sum(ctx_len) + sum(q_len)
    assert orc.step_position(130, 9, 0) == 139 and orc.step_position(5, 3, 3) == 11


# ------------------------------------------------------------------ independence of questions
def test_answers_do_not_depend_on_question_order_or_duplicates():
    from paper_2609_05707_b200 import workloads as W
    geom = W.Geometry(1, 4, 2, 16, 1e4)
    wl = W.custom_workload("t", geom, 77, [9], [3], [2, 5, 3], [2, 2, 2])
    outs = {k: orc.attend_tuple(wl, 0, k, 1, 0, 1) for k in range(3)}

    class Permuted:
        """Same raw tensors, questions presented in another order (1, 2, 0) plus a duplicate of 1."""
        geom = wl.geom
        order = [1, 2, 0, 1]

        def ctx_kv(self, b, layer): return wl.ctx_kv(b, layer)
        def question_kv(self, k, layer): return wl.question_kv(self.order[k], layer)
        def step_kv(self, s, layer, q): return wl.step_kv(s, layer, [self.order[i] for i in q])
        def step_q(self, s, layer, q): return wl.step_q(s, layer, [self.order[i] for i in q])

    pw = Permuted()
    for newk, oldk in enumerate(pw.order):
        np.testing.assert_array_equal(orc.attend_tuple(pw, 0, newk, 1, 0, 1), outs[oldk])


# ------------------------------------------------------------------ the per-tuple driver
def _dense_rows_of_step(wl, b, s, layer):
    """Dense-mask formulation of prompt b at decode step s: for every query head, the rows of the answer tokens fed at
    step s, computed by dense_attend over the whole stacked sequence.  The stacked sequence is assembled here from the
    workload's raw accessors, independently of attend_tuple; the KV head of a query head is chosen by an explicit
    repeat of every KV head G times (the order of HF `repeat_kv`: query heads [g*G, (g+1)*G) share KV head g)."""
    g = wl.geom
    G = g.n_q_heads // g.n_kv_heads
    L = int(wl.ctx_len[b])
    k0, k1 = int(wl.q_begin[b]), int(wl.q_begin[b + 1])
    q_lens = [int(wl.q_len[k]) for k in range(k0, k1)]
    # answer tokens in the cache after the append of step s: a question with stop step e has fed min(e, s + 1) tokens
    n_answer = [min(int(wl.stop[k]), s + 1) for k in range(k0, k1)]
    pos, ctx, qtn, tag = orc.stacked_sequence(0, [L], [q_lens], [n_answer])
    mask = orc.dense_mask(pos, ctx, qtn)
    n = len(pos)
    kc, vc = wl.ctx_kv(b, layer)
    K = np.zeros((n, g.n_kv_heads, g.head_dim))
    V = np.zeros_like(K)
    Q = np.zeros((n, g.n_q_heads, g.head_dim))
    rows = {}
    for i, (kind, _, kk, idx) in enumerate(tag):
        k = k0 + kk
        if kind == "c":
            K[i], V[i] = kc[idx].double().numpy(), vc[idx].double().numpy()
        elif kind == "x":
            kq, vq = wl.question_kv(k, layer)
            K[i], V[i] = kq[idx].double().numpy(), vq[idx].double().numpy()
        else:
            ka, va = wl.step_kv(idx, layer, [k])
            K[i], V[i] = ka[0].double().numpy(), va[0].double().numpy()
            if idx == s:
                Q[i] = wl.step_q(s, layer, [k])[0].double().numpy()
                rows[k] = i
    K_rep, V_rep = np.repeat(K, G, axis=1), np.repeat(V, G, axis=1)  # [n, Hq, D]
    out = {}
    for h in range(g.n_q_heads):
        o = orc.dense_attend(Q[:, h], K_rep[:, h], V_rep[:, h], pos, mask, g.rope_theta)
        for k, i in rows.items():
            out[(k, h)] = o[i]
    return out


def test_attend_tuple_equals_the_dense_mask_formulation():
    # Sec. 4.2: the IPPD output of an answer token under the dense mask over the stacked sequence equals the output of
    # its triplet prompted alone.  attend_tuple assembles the standalone prompt; the dense side is assembled above from
    # the raw accessors without it.  Two prompts, G = 2 and G = 4, ragged question lengths and stop steps, steps >= 2:
    # a wrong number of answer tokens (range(s) for range(s + 1)), a KV-head slice shifted by one query head, a wrong
    # question's tokens or a wrong step's query each break the agreement.
    from paper_2609_05707_b200 import workloads as W
    for hq, hkv in [(4, 2), (8, 2)]:
        wl = W.custom_workload("pin", W.Geometry(2, hq, hkv, 16, 1e4), 77, [9, 5], [3, 2], [2, 4, 1, 3, 2],
                               [4, 1, 3, 2, 4])
        G = hq // hkv
        checked = 0
        for s in range(wl.n_steps):
            act = wl.active(s)
            for b in range(wl.n_prompts):
                dense = _dense_rows_of_step(wl, b, s, layer=1)
                mine = [int(k) for k in act if wl.prompt_of[k] == b]
                assert sorted({k for k, _ in dense}) == mine  # exactly the active questions have a row at step s
                for k in mine:
                    for kv_head in range(hkv):
                        got = orc.attend_tuple(wl, b, k, s, 1, kv_head)
                        for j in range(G):
                            np.testing.assert_allclose(got[j], dense[(k, kv_head * G + j)], atol=1e-12, rtol=0)
                            checked += 1
        assert checked == int(wl.stop.sum()) * hq


def _dense_rows_of_batch_step(wl, s, layer):
    """The whole batch as ONE stacked sequence [p, c_1, x_11, .., c_2, x_21, ..] (Sec. 4.1): the shared instruction p
    with context id 0, every prompt of the batch as one context of the stacked prompt, then the answer tokens.  Returns
    the dense-mask attention rows of the answer tokens fed at step s, per query head, assembled from the raw accessors
    without attend_tuple."""
    g = wl.geom
    G = g.n_q_heads // g.n_kv_heads
    P = wl.shared_len
    B = wl.n_prompts
    q_lens = [[int(wl.q_len[k]) for k in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1]))] for b in range(B)]
    n_answer = [[min(int(wl.stop[k]), s + 1) for k in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1]))]
                for b in range(B)]
    pos, ctx, qtn, tag = orc.stacked_sequence(P, [int(v) for v in wl.ctx_len], q_lens, n_answer)
    mask = orc.dense_mask(pos, ctx, qtn)
    n = len(pos)
    K = np.zeros((n, g.n_kv_heads, g.head_dim))
    V = np.zeros_like(K)
    Q = np.zeros((n, g.n_q_heads, g.head_dim))
    kp, vp = wl.shared_kv(layer) if P else (None, None)
    rows = {}
    for i, (kind, j, kk, idx) in enumerate(tag):
        k = int(wl.q_begin[j]) + kk
        if kind == "p":
            K[i], V[i] = kp[idx].double().numpy(), vp[idx].double().numpy()
        elif kind == "c":
            kc, vc = wl.ctx_kv(j, layer, t0=idx, t1=idx + 1)
            K[i], V[i] = kc[0].double().numpy(), vc[0].double().numpy()
        elif kind == "x":
            kq, vq = wl.question_kv(k, layer)
            K[i], V[i] = kq[idx].double().numpy(), vq[idx].double().numpy()
        else:
            ka, va = wl.step_kv(idx, layer, [k])
            K[i], V[i] = ka[0].double().numpy(), va[0].double().numpy()
            if idx == s:
                Q[i] = wl.step_q(s, layer, [k])[0].double().numpy()
                rows[k] = i
    K_rep, V_rep = np.repeat(K, G, axis=1), np.repeat(V, G, axis=1)
    out = {}
    for h in range(g.n_q_heads):
        o = orc.dense_attend(Q[:, h], K_rep[:, h], V_rep[:, h], pos, mask, g.rope_theta)
        for k, i in rows.items():
            out[(k, h)] = o[i]
    return out


@pytest.mark.parametrize("shared_len", [0, 6])
def test_attend_tuple_equals_one_stacked_prompt_with_several_contexts(shared_len):
    # Sec. 4.1 / 4.4: several contexts stacked in one prompt behind a shared instruction p (context id 0, attended by
    # everybody; M_ctx keeps the contexts apart).  The standalone prompt of a triplet is (p, c_j, x_jk, answers); its
    # output must equal the dense-mask row over the whole stacked batch.  A wrong position offset for p, a context
    # leaking into another context's questions, or p missing from the standalone prompt each break the agreement.
    from paper_2609_05707_b200 import workloads as W
    wl = W.custom_workload("pin3", W.Geometry(1, 4, 2, 16, 1e4), 78, [5, 0, 7], [2, 1, 2], [2, 3, 1, 2, 4],
                           [3, 2, 1, 3, 2], shared_len=shared_len)
    checked = 0
    for s in range(wl.n_steps):
        dense = _dense_rows_of_batch_step(wl, s, 0)
        act = [int(k) for k in wl.active(s)]
        assert sorted({k for k, _ in dense}) == act
        for k in act:
            for kv_head in range(2):
                got = orc.attend_tuple(wl, int(wl.prompt_of[k]), k, s, 0, kv_head)
                for j in range(2):
                    np.testing.assert_allclose(got[j], dense[(k, kv_head * 2 + j)], atol=1e-12, rtol=0)
                    checked += 1
    assert checked == int(wl.stop.sum()) * 4


def test_layout_with_a_shared_instruction():
    # closed forms of Sec. 4.1 with an instruction of P tokens: p -> [0, P), c_b -> [P, P + L_b), x_k -> from P + L_b
    lay = orc.layout([3, 2], [1, 2], [2, 1, 3], [4, 4, 4], 128, 128, shared_len=5)
    assert lay["hdr_pos_virt"].tolist() == [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 5, 6, 7, 7, 8, 9]
    assert lay["hdr_ctx_id"].tolist() == [0] * 5 + [1] * 5 + [2] * 6
    assert lay["hdr_qtn_id"].tolist() == [0] * 5 + [0, 0, 0, 1, 1] + [0, 0, 2, 3, 3, 3]
    assert lay["hdr_begin"].tolist() == [5, 10, 16] and lay["ctx_tile_off"].tolist() == [1, 2, 3]
    assert orc.step_position(3, 2, 4, shared_len=5) == 14


# ------------------------------------------------------------------ prefill of the stacked header
def test_standalone_prefill_matches_library_causal_sdpa():
    # library routine: torch SDPA with is_causal on an independently written complex-number RoPE
    T, H, D, theta = 37, 3, 16, 1e4
    r = np.random.default_rng(5)
    k_raw, v_raw, q_raw = r.standard_normal((T, D)), r.standard_normal((T, D)), r.standard_normal((T, H, D))

    def crope(x, pos):
        z = x[..., : D // 2] + 1j * x[..., D // 2:]
        w = np.exp(1j * pos * theta ** (-np.arange(D // 2) / (D / 2)))
        zz = z * w
        return np.concatenate([zz.real, zz.imag], axis=-1)

    k = np.stack([crope(k_raw[i], i) for i in range(T)])
    q = np.stack([crope(q_raw[i], i) for i in range(T)])  # [T, H, D]
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q).permute(1, 0, 2)[None], torch.tensor(k)[None, None].expand(1, H, T, D),
        torch.tensor(v_raw)[None, None].expand(1, H, T, D), is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(orc.standalone_prefill(k_raw, v_raw, q_raw, theta), want, atol=1e-12)
    # its last row is the decode definition
    np.testing.assert_allclose(orc.standalone_prefill(k_raw, v_raw, q_raw, theta)[-1],
                               orc.standalone_attend(k_raw, v_raw, q_raw[-1], theta), atol=1e-12)


@pytest.mark.parametrize("shared_len", [0, 4])
def test_prefill_tuple_equals_header_rows_of_the_dense_formulation(shared_len):
    # Sec. 4.1: under the dense mask a context token sees p and its own context causally, a question token sees p,
    # its context and its own question prefix.  The header rows of dense_attend over the stacked sequence of the whole
    # batch must equal the rows of the standalone prompts (p, c_b) and (p, c_b, x_k).
    from paper_2609_05707_b200 import workloads as W
    wl = W.custom_workload("pin4", W.Geometry(1, 4, 2, 16, 1e4), 79, [5, 3], [2, 1], [2, 3, 4], [1, 1, 1],
                           shared_len=shared_len)
    g, G, P = wl.geom, 2, wl.shared_len
    q_lens = [[2, 3], [4]]
    pos, ctx, qtn, tag = orc.stacked_sequence(P, [5, 3], q_lens, [[0, 0], [0]])
    mask = orc.dense_mask(pos, ctx, qtn)
    n = len(pos)
    K, V, Q = np.zeros((n, 2, 16)), np.zeros((n, 2, 16)), np.zeros((n, 4, 16))
    for i, (kind, j, kk, idx) in enumerate(tag):
        k = int(wl.q_begin[j]) + kk
        if kind == "p":
            src = (wl.shared_kv(0), wl.shared_q(0))
        elif kind == "c":
            src = (wl.ctx_kv(j, 0), wl.ctx_q(j, 0))
        else:
            src = (wl.question_kv(k, 0), wl.question_q(k, 0))
        K[i], V[i], Q[i] = src[0][0][idx].double().numpy(), src[0][1][idx].double().numpy(), src[1][idx].double().numpy()
    dense = np.stack([orc.dense_attend(Q[:, h], np.repeat(K, G, axis=1)[:, h], np.repeat(V, G, axis=1)[:, h], pos, mask,
                                       g.rope_theta) for h in range(4)], axis=1)  # [n, Hq, D]
    for kv_head in range(2):
        hs = slice(kv_head * G, (kv_head + 1) * G)
        for b in range(2):
            rows_c = [i for i, t in enumerate(tag) if t[0] == "c" and t[1] == b]
            rows_p = [i for i, t in enumerate(tag) if t[0] == "p"]
            got = orc.prefill_tuple(wl, b, None, 0, kv_head)
            np.testing.assert_allclose(got, dense[rows_p + rows_c][:, hs], atol=1e-12, rtol=0)
            for k in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1])):
                rows_x = [i for i, t in enumerate(tag) if t[0] == "x" and t[1] == b and t[2] == k - int(wl.q_begin[b])]
                np.testing.assert_allclose(orc.prefill_tuple(wl, b, k, 0, kv_head), dense[rows_x][:, hs], atol=1e-12,
                                           rtol=0)


# --------------------------------------------------------------------------- the 8-bit cache variant
def _all_e4m3_values():
    """Every finite e4m3 number from the bit fields (1-4-3, bias 7, subnormals, S.1111.111 is not a number)."""
    vals = []
    for code in range(256):
        sgn = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 15 and m == 7:
            continue
        vals.append(sgn * (2.0 ** -6 * m / 8 if e == 0 else 2.0 ** (e - 7) * (1 + m / 8)))
    return np.array(sorted(set(vals)))


def test_quantize_e4m3_hand_values():
    # spacing 1/32 in [1/4, 1/2): 0.3 -> 10/32; 2^-5 in [1/8, 1/4); ties go to the even mantissa; 448 is the largest
    x = np.array([0.3, 0.2, 1.0625, 1.1875, 17.0, 19.0, 300.0, 447.0, 464.0, 1e6, -0.3, 0.0, 2.0 ** -10, 3 * 2.0 ** -10,
                  0.0009])
    want = np.array([0.3125, 0.203125, 1.0, 1.25, 16.0, 20.0, 288.0, 448.0, 448.0, 448.0, -0.3125, 0.0, 0.0,
                     2.0 ** -8, 0.0])
    np.testing.assert_array_equal(orc.quantize_e4m3(x), want)


def test_quantize_e4m3_is_the_nearest_code_by_enumeration():
    codes = _all_e4m3_values()
    assert codes.size == 253 and codes.max() == 448.0 and codes[codes > 0].min() == 2.0 ** -9  # +-126 and one zero
    np.testing.assert_array_equal(orc.quantize_e4m3(codes), codes)  # fixed points
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(size=4000), rng.normal(size=2000) * 40, rng.normal(size=2000) * 0.01,
                        rng.uniform(-460, 460, size=2000)])
    q = orc.quantize_e4m3(x)
    d = np.abs(x[:, None] - codes[None, :])
    best = d.min(axis=1)
    assert np.all(np.isin(q, codes))
    np.testing.assert_allclose(np.abs(x - q), best, rtol=0, atol=1e-15)  # no code is nearer
    # exact midpoints between neighbouring codes go to the code with the even mantissa (the even multiple of the
    # smaller code's spacing)
    mid = (codes[:-1] + codes[1:]) / 2
    qm = orc.quantize_e4m3(mid)
    lo, hi = codes[:-1], codes[1:]
    step = np.minimum(np.abs(hi - lo), 2.0 ** 5)
    k_lo = np.rint(np.abs(lo) / step)
    even_is_lo = (k_lo % 2 == 0)
    # around zero and across binades the rule is the same in units of the finer spacing
    np.testing.assert_array_equal(qm, np.where(even_is_lo, lo, hi))


def test_quantize_e4m3_equals_the_library_cast():
    rng = np.random.default_rng(6)
    x = np.concatenate([rng.normal(size=20000), rng.normal(size=5000) * 30, rng.normal(size=5000) * 0.02])
    x = x[np.abs(x) < 440].astype(np.float32)  # the library's cast does not saturate the same way beyond the range
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(orc.quantize_e4m3(x.astype(np.float64)), lib)


def test_attend_e4m3_is_plain_attention_over_the_quantised_cache():
    rng = np.random.default_rng(8)
    T, D, H, theta = 37, 64, 4, 1e4
    k_raw, v_raw, q_raw = rng.normal(size=(T, D)), rng.normal(size=(T, D)), rng.normal(size=(H, D))
    got = orc.standalone_attend(k_raw, v_raw, q_raw, theta, kv_e4m3=True)
    # independent route: the library's float8 cast of the rotated keys and of the values, then torch SDPA's last row
    k8 = torch.from_numpy(orc.rope(k_raw, np.arange(T), theta).astype(np.float32)).to(torch.float8_e4m3fn).double()
    v8 = torch.from_numpy(v_raw.astype(np.float32)).to(torch.float8_e4m3fn).double()
    q = torch.from_numpy(orc.rope(q_raw, np.full(H, T - 1), theta))
    want = torch.nn.functional.scaled_dot_product_attention(q[None], k8[None], v8[None])[0].numpy()
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)
    # and it differs from the unquantised result by what 3 mantissa bits cost, not by more
    exact = orc.standalone_attend(k_raw, v_raw, q_raw, theta)
    err = np.abs(got - exact).max() / np.sqrt((exact ** 2).mean())
    assert 1e-3 < err < 0.5


def test_prefill_e4m3_last_row_is_the_e4m3_decode_row():
    rng = np.random.default_rng(9)
    T, D, H, theta = 21, 64, 2, 1e4
    k_raw, v_raw, q_raw = rng.normal(size=(T, D)), rng.normal(size=(T, D)), rng.normal(size=(T, H, D))
    full = orc.standalone_prefill(k_raw, v_raw, q_raw, theta, kv_e4m3=True)
    for t in (0, 5, T - 1):  # row t of the prefill is the decode row of the prompt cut after token t
        row = orc.standalone_attend(k_raw[:t + 1], v_raw[:t + 1], q_raw[t], theta, kv_e4m3=True)
        np.testing.assert_allclose(full[t], row, rtol=1e-10, atol=1e-12)
