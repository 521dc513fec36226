"""The host-buffer entry points (blocking and pipelined) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, gate, oracle_step  # noqa: E402


def _workload():
    # two prompts, ragged question counts and lengths, stops that differ so that the active set shrinks
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    return W.custom_workload("host-steps", geom, 31, [300, 77], [3, 2], [9, 130, 20, 7, 33], [6, 4, 6, 3, 5])


def _host_inputs(run, wl, s):
    act = wl.active(s)
    q, k, v = run.step_inputs(s, act)
    return act, tuple(t.cpu().pin_memory() for t in (q, k, v))


def _check_step(wl, s, act, out, cache, what):
    G = wl.geom.group
    got, want = [], []
    for layer in range(wl.geom.n_layers):
        for h in range(wl.geom.n_kv_heads):
            ref = oracle_step(wl, s, layer, h, cache)
            for i, k in enumerate(act):
                got.append(out[layer, i, h * G:(h + 1) * G])
                want.append(ref[int(k)])
    gate(np.stack(got), np.stack(want), f"{what} step {s}")


@pytest.mark.parametrize("pipelined", [False, True])
def test_host_steps_match_the_oracle(pipelined):
    wl = _workload()
    g = wl.geom
    run = PoisonedRunner(wl, out_dtype=B.F32)
    run.load_header()
    n_steps = wl.n_steps
    amax = max(len(wl.active(s)) for s in range(n_steps))
    slots = 2 if pipelined else 1
    stage = run.alloc_bytes(slots * run.layout.step_stage_bytes(amax) + 256, "stage")
    stage.fill_(0xFF)
    steps = [_host_inputs(run, wl, s) for s in range(n_steps)]
    outs = [torch.full((g.n_layers, len(a), g.n_q_heads, g.head_dim), float("nan")).pin_memory() for a, _ in steps]
    for s, (act, (hq, hk, hv)) in enumerate(steps):
        idx = np.full(len(act), s, dtype=np.int32)
        if pipelined:
            run.layout.decode_step_host_async(act, idx, hq, hk, hv, outs[s], stage, run.workspace, run.stream)
        else:
            run.layout.decode_step_host(act, idx, hq, hk, hv, outs[s], stage, run.workspace, run.stream)
    if pipelined:
        run.layout.host_steps_wait(run.stream)
    run.check()
    cache = {}
    for s, (act, _) in enumerate(steps):
        _check_step(wl, s, act, outs[s].numpy(), cache, "pipelined" if pipelined else "blocking")


def test_pipelined_steps_equal_blocking_steps_bit_for_bit():
    wl = _workload()
    g = wl.geom
    results = []
    for pipelined in (False, True):
        run = PoisonedRunner(wl, out_dtype=B.F32)
        run.load_header()
        amax = max(len(wl.active(s)) for s in range(wl.n_steps))
        stage = run.alloc_bytes(2 * run.layout.step_stage_bytes(amax), "stage")
        outs = []
        for s in range(wl.n_steps):
            act, (hq, hk, hv) = _host_inputs(run, wl, s)
            out = torch.empty((g.n_layers, len(act), g.n_q_heads, g.head_dim)).pin_memory()
            idx = np.full(len(act), s, dtype=np.int32)
            fn = run.layout.decode_step_host_async if pipelined else run.layout.decode_step_host
            fn(act, idx, hq, hk, hv, out, stage, run.workspace, run.stream)
            outs.append(out)
        run.layout.host_steps_wait(run.stream)
        run.check()
        results.append([o.numpy().copy() for o in outs])
    for a, b in zip(*results):
        assert np.array_equal(a, b)


def test_pipelined_step_rejects_a_one_slot_staging_buffer():
    wl = _workload()
    run = PoisonedRunner(wl, out_dtype=B.F32)
    run.load_header()
    act, (hq, hk, hv) = _host_inputs(run, wl, 0)
    g = wl.geom
    out = torch.empty((g.n_layers, len(act), g.n_q_heads, g.head_dim)).pin_memory()
    stage = torch.empty(run.layout.step_stage_bytes(len(act)), dtype=torch.uint8, device=run.device)
    with pytest.raises(B.IppdError) as e:
        run.layout.decode_step_host_async(act, np.zeros(len(act), dtype=np.int32), hq, hk, hv, out, stage,
                                          run.workspace, run.stream)
    assert e.value.code == B.ERR_INVALID_ARG
