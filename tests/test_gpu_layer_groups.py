"""Layer-range calls and steps with more than 64 active questions against the oracle, through the C ABI."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, compare_step  # noqa: E402


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("layers_per_call", [1, 2])
def test_layer_groups_match_the_oracle(kernel, layers_per_call):
    # five layers in groups of one or two (the last group of the latter is ragged): the first STEP append of a step
    # carries the descriptor upload, the later ones and the attention calls of every group find it on the device
    geom = W.Geometry(5, 8, 2, 128, 5e5)
    wl = W.custom_workload("groups", geom, 41, [260, 31], [3, 2], [12, 7, 130, 9, 20], [4, 3, 4, 2, 4])
    run = PoisonedRunner(wl, out_dtype=B.F32, kernel=kernel, layers_per_call=layers_per_call)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, range(geom.n_layers), range(geom.n_kv_heads), cache, f"groups of {layers_per_call}")


@pytest.mark.parametrize("kernel", [1, 2])
def test_more_than_64_active_questions(kernel):
    # 70 + 3 questions: the active list no longer fits the append's kernel parameters (separate descriptor upload),
    # and the first prompt's rows span three 128-row blocks that all stream the same context
    geom = W.Geometry(1, 8, 2, 64, 1e4)
    r = np.random.default_rng(7)
    qc = [70, 3]
    ql = r.integers(1, 20, sum(qc)).tolist()
    stop = r.integers(1, 4, sum(qc)).tolist()
    stop[0] = 3
    wl = W.custom_workload("many", geom, 17, [150, 40], qc, ql, stop)
    run = PoisonedRunner(wl, out_dtype=B.F32, kernel=kernel)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, [0], range(geom.n_kv_heads), cache, "many questions")


def test_read_probe_streams_the_step_and_changes_nothing():
    # the measuring aid walks the same tile list as the attention kernel and discards it: no output, no error, the
    # cache untouched, and the step it was declared for still computes correctly afterwards
    import torch
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    wl = W.custom_workload("probe", geom, 43, [700, 130], [5, 40], [20] * 45, [3] * 45)
    run = PoisonedRunner(wl, out_dtype=B.F32)
    run.load_header()
    run.run_step(0)
    snapshot = run.cache.clone()
    act = wl.active(1)
    run.layout.begin_step(act, np.full(len(act), 1, dtype=np.int32), run.stream)
    for _ in range(3):
        run.layout.read_probe(0, geom.n_layers, run.stream)
    run.check()
    assert torch.equal(snapshot, run.cache)
    t = run.layout.host_time_read()
    assert t["steps"] >= 1 and t["begin_step_us"] > 0
    cache = {}
    compare_step(run, 1, range(2), range(2), cache, "after the probe")
