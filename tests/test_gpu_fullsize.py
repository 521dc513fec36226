"""Full-size configurations in the launch configuration bench.py times (all layers in one call), checked on sampled
outputs the oracle computes one by one.

A tuple is one (prompt, question, step, layer, query head) output row.  Every configuration is sampled on at least 4096
tuples, stratified: the first step, a step just before a question's stop step and the last step; the first and the
last layer and KV head (plus one in between); in every prompt the first, the last, the shortest and the longest active
question and every question about to stop.  C2 is also checked on EVERY tuple of one whole (layer, step)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, gate, oracle_step  # noqa: E402

MIN_TUPLES = 4096


def pick_stratified(wl, act, s, per_prompt):
    """First, last, shortest and longest active question of every prompt, the questions whose last step this is, and
    evenly spaced others up to `per_prompt` per prompt."""
    out = []
    for b in range(wl.n_prompts):
        mine = [int(k) for k in act if wl.prompt_of[k] == b]
        if not mine:
            continue
        lens = wl.q_len[mine]
        chosen = {mine[0], mine[-1], mine[int(np.argmin(lens))], mine[int(np.argmax(lens))]}
        chosen |= {k for k in mine if wl.stop[k] == s + 1}
        chosen = set(sorted(chosen)[:per_prompt])  # a whole batch stopping at once is not a reason to check them all
        chosen |= {mine[0], mine[-1], mine[int(np.argmin(lens))], mine[int(np.argmax(lens))]}
        rest = [k for k in mine if k not in chosen]
        want = max(0, per_prompt - len(chosen))
        if want and rest:
            chosen |= set(rest[:: max(1, len(rest) // want)][:want])
        out += sorted(chosen)
    return out


def run_and_sample(name, check, per_prompt, kernel=0, full_layer_step=None, kv_dtype=B.KV_BF16):
    """check: {step: [(layer, kv head), ...]}.  Returns the number of tuples compared."""
    wl = W.make_workload(name)
    G = wl.geom.group
    run = PoisonedRunner(wl, kernel=kernel, kv_dtype=kv_dtype)
    run.load_header()
    # the K/V of every step go into the cache first (a token's slot depends only on its question and step index, and a
    # step reads no slot beyond its own), then only the sampled steps are run; each of them appends its own token again
    run.append_all_steps()
    ctx_cache, step_cache = {}, {}
    n_tuples = 0
    for s in sorted(check):
        act, out = run.run_step(s)
        run.check()
        rows = {int(k): i for i, k in enumerate(act)}
        for layer, head in check[s]:
            everything = full_layer_step == (layer, s)
            qids = [int(k) for k in act] if everything else pick_stratified(wl, act, s, per_prompt)
            ref = oracle_step(wl, s, layer, head, ctx_cache, step_cache, qids, kv_e4m3=kv_dtype == B.KV_E4M3)
            o = out[layer, :, head * G:(head + 1) * G].float().cpu().numpy()
            got = np.stack([o[rows[k]] for k in qids])
            want = np.stack([ref[k] for k in qids])
            gate(got, want, f"{name} step {s} layer {layer} head {head}")
            n_tuples += got.shape[0] * G
    run.check()
    del run
    torch.cuda.empty_cache()
    return n_tuples


def _layer_heads(wl, extra=()):
    g = wl.geom
    last_l, last_h = g.n_layers - 1, g.n_kv_heads - 1
    return [(0, 0), (0, last_h), (last_l, 0), (last_l, last_h), (g.n_layers // 2, g.n_kv_heads // 2)] + list(extra)


def _steps(wl, extra=()):
    last = int(wl.stop.max()) - 1
    srt = np.sort(wl.stop)
    before_eos = [int(srt[len(srt) * i // 4]) - 1 for i in (1, 2, 3)]  # last steps of the quartile questions
    return sorted({0, last, *before_eos, *extra})


def test_c2_full_size_sampled_warp_level_path():
    # the earlier mma.sync path (IPPD_OPT_KERNEL = 1) on a thinner sample
    lh = [(0, 0), (17, 5), (31, 7)]
    run_and_sample("C2", {0: lh, 40: lh}, per_prompt=16, kernel=1)


def test_c2_full_size_sampled(kernel=2):
    wl = W.make_workload("C2")
    # C2 has no stop steps: four steps spread over the schedule; every KV head of layer 17 at step 63 (= every tuple
    # of that layer and step)
    lh = _layer_heads(wl, [(5, 1), (9, 6), (23, 2), (28, 5), (2, 3), (30, 4), (12, 7)])
    check = {0: lh, 31: lh, 95: lh, 127: lh,
             63: lh + [(17, h) for h in range(wl.geom.n_kv_heads)]}
    n = run_and_sample("C2", check, per_prompt=16, kernel=kernel, full_layer_step=(17, 63))
    assert n >= MIN_TUPLES, n


def test_c3_full_size_sampled():
    wl = W.make_workload("C3")
    lh = _layer_heads(wl, [(7, 5), (19, 2), (26, 6), (3, 3), (29, 1), (14, 7), (22, 0)])
    n = run_and_sample("C3", {s: lh for s in _steps(wl, [7, 40])}, per_prompt=32)
    assert n >= MIN_TUPLES, n


def test_c2_full_size_sampled_e4m3_cache():
    # the 8-bit cache variant in the bench's launch configuration, against the oracle over the quantised cache
    wl = W.make_workload("C2")
    lh = _layer_heads(wl, [(5, 1), (9, 6), (23, 2), (28, 5)])
    check = {0: lh, 63: lh + [(17, h) for h in range(wl.geom.n_kv_heads)], 127: lh}
    n = run_and_sample("C2", check, per_prompt=16, full_layer_step=(17, 63), kv_dtype=B.KV_E4M3)
    assert n >= MIN_TUPLES // 2, n


def test_c3_full_size_sampled_e4m3_cache():
    wl = W.make_workload("C3")
    lh = _layer_heads(wl, [(7, 5), (19, 2), (26, 6)])
    last = int(wl.stop.max()) - 1
    n = run_and_sample("C3", {s: lh for s in (0, 40, last)}, per_prompt=32, kv_dtype=B.KV_E4M3)
    assert n >= 1024, n


def test_c4_full_size_sampled():
    wl = W.make_workload("C4")
    n = run_and_sample("C4", {0: _layer_heads(wl), 127: _layer_heads(wl)[:4]}, per_prompt=5)
    assert n >= MIN_TUPLES, n


def test_c5_full_size_sampled():
    wl = W.make_workload("C5")
    lh = [(0, 0), (79, 7), (40, 3)]
    n = run_and_sample("C5", {s: lh for s in _steps(wl)}, per_prompt=20)
    assert n >= MIN_TUPLES, n


def test_s1_full_size_sampled():
    # second workload family (shapes of the paper's dataset table): long contexts, many questions, short answers
    wl = W.make_workload("S1")
    n = run_and_sample("S1", {s: _layer_heads(wl) for s in _steps(wl, [5])}, per_prompt=12)
    assert n >= MIN_TUPLES, n


def test_s2_full_size_sampled():
    wl = W.make_workload("S2")
    lh = _layer_heads(wl, [(7, 5), (19, 2), (26, 6), (3, 3), (29, 1), (14, 7), (22, 0), (10, 4)])
    n = run_and_sample("S2", {s: lh for s in _steps(wl, [3])}, per_prompt=12)
    assert n >= MIN_TUPLES, n


@pytest.mark.parametrize("name", ["SWEEP-L2048-Q1", "SWEEP-L2048-Q32", "SWEEP-L16384-Q1", "SWEEP-L16384-Q32"])
def test_sweep_corners_sampled(name):
    # the four corners of the questions-per-context x context-length sweep (the axes of the paper's ablations)
    wl = W.make_workload(name)
    run_and_sample(name, {0: [(0, 0), (31, 7)], 15: [(0, 0), (16, 3), (31, 7)]}, per_prompt=8)
