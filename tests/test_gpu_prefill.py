"""Prefill of the stacked header under the IPPD mask (paper Sec. 4, Sec. 4.1 header rows, App. A.2) against the
oracle, in which every header row is the row of its own standalone causal prompt."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, compare_step, gate, orc  # noqa: E402


def _header_index(wl):
    """Header offsets: (first token of the instruction = 0, first context token of each prompt, first token of each
    question), in the order of the layout's hdr_* tables."""
    ctx0, q0 = [], {}
    t = wl.shared_len
    for b in range(wl.n_prompts):
        ctx0.append(t)
        t += int(wl.ctx_len[b])
        for k in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1])):
            q0[k] = t
            t += int(wl.q_len[k])
    return ctx0, q0, t


def _compare_header(wl, out, layers, heads, ctx_rows=None, questions=None, what="prefill", kv_e4m3=False):
    """out: [n_layers, n_hdr, Hq, D] numpy.  ctx_rows: {b: positions inside (instruction + context)} or None = all;
    questions: ids or None = all."""
    G, P = wl.geom.group, wl.shared_len
    ctx0, q0, n_hdr = _header_index(wl)
    assert out.shape[1] == n_hdr
    got, want = [], []
    for layer in layers:
        for h in heads:
            hs = slice(h * G, (h + 1) * G)
            for b in range(wl.n_prompts):
                rows = None if ctx_rows is None else ctx_rows.get(b, [])
                if rows is not None and len(rows) == 0:
                    continue
                Lb = int(wl.ctx_len[b])
                if P + Lb == 0:
                    continue  # no instruction and an empty context: the prompt has question rows only
                ref = orc.prefill_tuple(wl, b, None, layer, h, kv_e4m3)  # rows of p and c_b
                pick = range(P + Lb) if rows is None else rows
                for r in pick:
                    if r < P:
                        if b == 0:  # the instruction's rows are the same in every prompt: check them once
                            got.append(out[layer, r, hs]); want.append(ref[r])
                    else:
                        got.append(out[layer, ctx0[b] + r - P, hs]); want.append(ref[r])
            for k in (range(wl.n_questions) if questions is None else questions):
                ref = orc.prefill_tuple(wl, int(wl.prompt_of[k]), int(k), layer, h, kv_e4m3)
                for j in range(int(wl.q_len[k])):
                    got.append(out[layer, q0[k] + j, hs]); want.append(ref[j])
    # rows that see only a handful of keys have outputs of size ~1: the absolute gate is stated for averages over
    # many keys, so the per-row relative gates carry those
    return gate(np.stack(got), np.stack(want), what, absolute=False)


@pytest.mark.parametrize("tiles_per_split", [0, 3, 1000])
def test_c1_prefill_every_header_row(tiles_per_split):
    wl = W.make_workload("C1")
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=tiles_per_split)
    out = run.prefill().cpu().numpy()
    run.check()
    _compare_header(wl, out, [0], range(wl.geom.n_kv_heads), what="C1 prefill")
    # the cache is now what the append calls would have produced: the decode steps match the oracle
    cache = {}
    for s in (0, 1, 17):
        if s > 1:
            for t in range(2, s):
                run.run_step(t)
        compare_step(run, s, [0], range(wl.geom.n_kv_heads), cache, "C1 decode after prefill")


@pytest.mark.parametrize("shared_len", [0, 130])
def test_ragged_prefill_every_header_row_and_cache_equals_appends(shared_len):
    # contexts of 0, 1, 127..129 and several tiles; questions of 1..140 tokens (longer than a cache tile); an
    # instruction that ends inside a tile
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    ctx = [0, 1, 127, 128, 129, 300]
    qc = [1, 2, 3, 2, 9, 40]
    r = np.random.default_rng(11)
    ql = r.integers(1, 30, sum(qc)).tolist()
    ql[5] = 140
    wl = W.custom_workload("prefill-ragged", geom, 71, ctx, qc, ql, [2] * sum(qc), shared_len=shared_len)
    ref_run = PoisonedRunner(wl, out_dtype=B.F32)
    ref_run.load_header()
    outs = []
    for lpc in (1, 2):
        run = PoisonedRunner(wl, out_dtype=B.F32)
        outs.append(run.prefill(layers_per_call=lpc).cpu().numpy())
        run.check()
        assert torch.equal(run.cache, ref_run.cache)
    _compare_header(wl, outs[0], range(2), range(2), what="ragged prefill")
    # two layers per call cut the tile sequence elsewhere: same rows within rounding
    rms = np.sqrt((outs[0].astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
    assert (np.abs(outs[1] - outs[0]) / rms).max() <= 3e-2
    cache = {}
    for s in range(2):
        compare_step(run, s, range(2), range(2), cache, "decode after prefill")


def test_c2_prefill_sampled():
    wl = W.make_workload("C2", n_layers=4)
    run = PoisonedRunner(wl)
    out = run.prefill(layers_per_call=2).float().cpu().numpy()
    run.check()
    rows = {0: [0, 1, 31, 32, 127, 128, 129, 255, 256, 1000, 1023, 1024, 2046, 2047]}
    _compare_header(wl, out, [0, 3], [0, 7], ctx_rows=rows, questions=[0, 7, 15], what="C2 prefill")
