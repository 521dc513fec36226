"""An instruction shared by every prompt of the batch (paper Sec. 4.1 stacked header [p, c_1, .., c_2, ..]; Sec. 4.4:
the instruction's K/V kept once for the whole batch): three levels of sharing, instruction -> context -> branch,
against the oracle, whose standalone prompts start with the instruction."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, compare_step, orc  # noqa: E402
from test_gpu_fullsize import run_and_sample, _layer_heads, _steps, MIN_TUPLES  # noqa: E402


@pytest.mark.parametrize("tiles_per_split", [0, 1000])
@pytest.mark.parametrize("shared_len", [1, 127, 128, 300])
def test_shared_instruction_every_tuple(shared_len, tiles_per_split):
    # instruction lengths around the tile edges; contexts of 0, a partial tile and several tiles; the instruction is
    # stored once (cache tiles from 0) and every row block's key sequence starts with it
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    r = np.random.default_rng(shared_len)
    qc = [3, 1, 40]
    nq = sum(qc)
    wl = W.custom_workload("shared", geom, 61, [200, 0, 77], qc, r.integers(1, 40, nq).tolist(),
                           r.integers(1, 5, nq).tolist(), shared_len=shared_len)
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=tiles_per_split)
    run.load_header()
    tabs = run.layout.layout_tables()
    assert tabs["n_shared_tokens"] == shared_len and tabs["ctx_tile_off"][0] == (shared_len + 127) // 128
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, range(2), range(2), cache, f"shared {shared_len}")


def test_mask_export_with_a_shared_instruction():
    wl = W.custom_workload("mask-shared", W.Geometry(1, 8, 2, 64, 1e4), 3, [5, 3], [3, 2], [2, 4, 1, 3, 2], [4] * 5,
                           shared_len=4)
    run = PoisonedRunner(wl)
    n_answer = [[3, 0, 2], [1, 4]]
    for b in range(2):
        got = run.layout.export_mask(b, n_answer[b]).astype(bool)
        k0 = int(wl.q_begin[b])
        qls = [int(v) for v in wl.q_len[k0:k0 + wl.q_count[b]]]
        # the instruction keeps context id 0 (ctx = 0 for p in the mask predicates), the prompt is context 1
        pos, ctx, qtn, tag = orc.stacked_sequence(4, [int(wl.ctx_len[b])], [qls], [n_answer[b]])
        np.testing.assert_array_equal(got, orc.dense_mask(pos, ctx, qtn))


def test_shared_instruction_is_refused_by_the_warp_level_path():
    wl = W.custom_workload("shared-k1", W.Geometry(1, 8, 2, 64, 1e4), 3, [5], [2], [2, 4], [2, 2], shared_len=4)
    run = PoisonedRunner(wl, kernel=1)
    with pytest.raises(B.IppdError) as e:
        run.layout.begin_step([0, 1], [0, 0], run.stream)
    assert e.value.code == B.ERR_INVALID_ARG


def test_s3_full_size_sampled():
    # twelve prompts behind a 2754-token instruction (shapes of the paper's few-shot workload)
    wl = W.make_workload("S3")
    n = run_and_sample("S3", {s: _layer_heads(wl) for s in _steps(wl)}, per_prompt=8)
    assert n >= MIN_TUPLES, n
