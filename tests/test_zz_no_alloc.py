"""The allocation-free attention entry point gives the same output as the ordinary one.

Some users of the library cannot allocate device memory where they run attention (a serving loop whose
allocator has handed everything out, a plug-in that must not allocate after start-up, a latency-critical
loop that cannot risk an allocation's implicit synchronisation), so they cannot pass a workspace.
ippd_decode_attention_static keeps the split-KV partials in an array built into the library instead.
This file is collected last so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner  # noqa: E402


def _one_step(run, s, use_static):
    wl, g = run.wl, run.wl.geom
    act = wl.active(s)
    q, k, v = run.step_inputs(s, act)
    out = torch.full((g.n_layers, len(act), g.n_q_heads, g.head_dim), float("nan"), dtype=torch.float32,
                     device=run.device)
    run.layout.begin_step(act, np.full(len(act), s, dtype=np.int32), run.stream)
    run.layout.append_kv(0, g.n_layers, B.APPEND_STEP, None, k, v, run.stream)
    if use_static:
        run.layout.decode_attention_static(0, g.n_layers, q, out, run.stream)
    else:
        run.layout.decode_attention(0, g.n_layers, q, out, run.workspace, run.stream)
    run.check()
    return out.cpu().numpy()


@pytest.mark.parametrize("kernel", [1, 2])
def test_static_scratch_entry_point_matches_workspace_entry_point(kernel):
    # several split-KV units per row block, so that the scratch (partials + merge) is really used
    wl = W.custom_workload("noalloc", W.Geometry(2, 8, 2, 128, 5e5), 21, [900, 300], [5, 18],
                           [20] * 23, [2] * 23)
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=2, kernel=kernel)
    run.load_header()
    for s in range(2):  # two calls in a row share the built-in array
        want = _one_step(run, s, use_static=False)
        got = _one_step(run, s, use_static=True)
        assert np.isfinite(got).all()
        # both entry points run the same kernels over the same partition of the keys; only the address of the
        # partials differs, so the results agree bit for bit (a tolerance would hide a slightly wrong scratch offset)
        assert np.array_equal(got, want), float(np.abs(got - want).max())


def test_static_scratch_entry_point_allocates_no_device_memory():
    # what the entry point is for: after a first (set-up) call, further calls leave the device's free memory and
    # torch's own allocation count exactly where they were
    wl = W.custom_workload("noalloc-mem", W.Geometry(2, 8, 2, 128, 5e5), 23, [900], [6], [20] * 6, [3] * 6)
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=2)
    run.load_header()
    g = wl.geom
    act = wl.active(0)
    q, k, v = run.step_inputs(0, act)
    out = run.alloc_out(len(act))
    idx = np.zeros(len(act), dtype=np.int32)
    run.layout.begin_step(act, idx, run.stream)
    run.layout.append_kv(0, g.n_layers, B.APPEND_STEP, None, k, v, run.stream)
    run.layout.decode_attention_static(0, g.n_layers, q, out, run.stream)  # set-up call
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for _ in range(3):
        run.layout.decode_attention_static(0, g.n_layers, q, out, run.stream)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == alloc0
    run.check()


def test_static_scratch_rejects_a_step_that_does_not_fit():
    # 40 layers x 8 KV heads x many single-tile units needs more than the built-in array holds (the unit-list
    # path; the persistent tensor-core path always needs less than the array)
    wl = W.custom_workload("toolarge", W.Geometry(40, 32, 8, 128, 5e5), 22, [128 * 70], [16], [8] * 16, [1] * 16)
    run = PoisonedRunner(wl, tiles_per_split=1, kernel=1)
    act = wl.active(0)
    g = wl.geom
    q = torch.zeros((g.n_layers, len(act), g.n_q_heads, g.head_dim), dtype=torch.bfloat16, device=run.device)
    out = torch.zeros_like(q)
    run.layout.begin_step(act, np.zeros(len(act), dtype=np.int32), run.stream)
    with pytest.raises(B.IppdError) as e:
        run.layout.decode_attention_static(0, g.n_layers, q, out, run.stream)
    assert e.value.code == B.ERR_CAPACITY and "bytes of scratch" in str(e.value)
    run.layout.decode_attention_static(0, 2, q[:2], out[:2], run.stream)  # two layers fit
    run.check()
