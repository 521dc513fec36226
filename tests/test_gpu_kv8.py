"""The 8-bit (e4m3) cache variant against the fp64 oracle over the quantised keys and values (needs a B200)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, compare_step, gate, oracle_step, orc  # noqa: E402


def _decode_e4m3(codes: np.ndarray) -> np.ndarray:
    """e4m3 bytes -> fp64 from the bit fields (1-4-3, bias 7, subnormals)."""
    c = codes.astype(np.int64)
    sgn = np.where(c & 0x80, -1.0, 1.0)
    e, m = (c >> 3) & 0xF, c & 0x7
    return sgn * np.where(e == 0, 2.0 ** -6 * m / 8, 2.0 ** (e - 7.0) * (1 + m / 8))


def test_c1_every_tuple_e4m3():
    wl = W.make_workload("C1")
    for out_dtype in (B.BF16, B.F32):
        r = PoisonedRunner(wl, out_dtype=out_dtype, kv_dtype=B.KV_E4M3)
        r.load_header()
        cache = {}
        for s in range(wl.n_steps):
            compare_step(r, s, [0], range(wl.geom.n_kv_heads), cache, "C1/e4m3")


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("tiles_per_split", [0, 1000])
def test_ragged_batch_with_stops_every_tuple_e4m3(tiles_per_split, fused):
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    ctx = [0, 1, 127, 128, 129, 700]
    qc = [1, 2, 3, 5, 17, 20]
    nq = sum(qc)
    r = np.random.default_rng(5)
    ql = r.integers(1, 40, nq).tolist()
    ql[3] = 120
    stop = r.integers(1, 14, nq).tolist()
    stop[3] = 14
    wl = W.custom_workload("ragged8", geom, 99, ctx, qc, ql, stop)
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=tiles_per_split, fused=fused, kv_dtype=B.KV_E4M3)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, range(2), range(2), cache, "ragged/e4m3")


@pytest.mark.parametrize("tiles_per_split", [0, 1000])
def test_branches_longer_than_a_cache_tile_e4m3(tiles_per_split):
    ql = [100, 127, 128, 129, 200, 255, 90, 260]
    wl = W.custom_workload("long-branches8", W.Geometry(1, 8, 2, 128, 5e5), 17, [300], [len(ql)], ql, [40] * len(ql))
    run = PoisonedRunner(wl, out_dtype=B.F32, tiles_per_split=tiles_per_split, kv_dtype=B.KV_E4M3)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        if s in (0, 1, 27, 28, 29, 39):
            compare_step(run, s, [0], range(2), cache, "long-branches/e4m3")
        else:
            run.run_step(s)
    run.check()


def test_cache_holds_the_nearest_e4m3_numbers():
    # the rotated keys and the values read back from the tiled cache are the oracle's e4m3 numbers; the kernel rotates
    # in fp32, so a value that lies within 2^-18 (relative) of the midpoint of two codes may land on either
    wl = W.custom_workload("rope8", W.Geometry(1, 4, 2, 128, 5e5), 11, [300], [2], [5, 9], [4, 4])
    run = PoisonedRunner(wl, kv_dtype=B.KV_E4M3)
    run.load_header()
    nbytes, _ = run.layout.cache_bytes()
    assert nbytes == 2 * run.layout.layout_tables()["n_tiles"] * 2 * 128 * 128  # one byte per element
    tiles = run.cache.view(1, 2, -1, 2, 16, 8, 8, 16)  # layer, head, tile, kv, tok/8, d/16, tok%8, d%16
    k_raw, v_raw = wl.ctx_kv(0, 0)
    for head in range(2):
        kt = tiles[0, head, :3, 0].permute(0, 1, 3, 2, 4).reshape(3 * 128, 128)[:300].cpu().numpy()
        vt = tiles[0, head, :3, 1].permute(0, 1, 3, 2, 4).reshape(3 * 128, 128)[:300].cpu().numpy()
        exact = orc.rope(k_raw[:, head].double().numpy(), np.arange(300), 5e5)
        want = orc.quantize_e4m3(exact)
        got = _decode_e4m3(kt)
        differ = got != want
        assert differ.mean() < 1e-3
        if differ.any():  # only at (near) ties, and then by one code: the other neighbour is as near
            assert np.all(np.abs(np.abs(got[differ] - exact[differ]) - np.abs(want[differ] - exact[differ]))
                          <= np.abs(exact[differ]) * 2.0 ** -18)
        np.testing.assert_array_equal(_decode_e4m3(vt), orc.quantize_e4m3(v_raw[:, head].double().numpy()))


def test_prefill_e4m3_every_header_row_then_decode():
    from test_gpu_prefill import _compare_header
    wl = W.make_workload("C1")
    run = PoisonedRunner(wl, out_dtype=B.F32, kv_dtype=B.KV_E4M3)
    out = run.prefill().cpu().numpy()
    run.check()
    _compare_header(wl, out, [0], range(wl.geom.n_kv_heads), what="C1 prefill/e4m3", kv_e4m3=True)
    cache = {}
    for s in (0, 1):
        compare_step(run, s, [0], range(wl.geom.n_kv_heads), cache, "C1 decode after prefill/e4m3")


def test_shared_instruction_e4m3():
    geom = W.Geometry(1, 8, 2, 128, 5e5)
    wl = W.custom_workload("shared8", geom, 5, [150, 40], [3, 2], [6, 9, 4, 7, 5], [5] * 5, shared_len=200)
    run = PoisonedRunner(wl, out_dtype=B.F32, kv_dtype=B.KV_E4M3)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, [0], range(2), cache, "shared/e4m3")


def test_the_cache_type_is_fixed_by_bind_and_needs_the_tensor_core_path():
    wl = W.make_workload("C1")
    run = PoisonedRunner(wl)
    with pytest.raises(B.IppdError):
        run.layout.set_option(B.OPT_KV_DTYPE, B.KV_E4M3)  # already bound
    geom = B.make_geometry(1, 8, 2, 64, 1e4)
    lay = B.Layout(geom, [16], [1], [4], [4])
    lay.set_option(B.OPT_KERNEL, 1)
    with pytest.raises(B.IppdError):
        lay.set_option(B.OPT_KV_DTYPE, B.KV_E4M3)
    lay.set_option(B.OPT_KERNEL, 2)
    full, _ = lay.cache_bytes()
    lay.set_option(B.OPT_KV_DTYPE, B.KV_E4M3)
    half, _ = lay.cache_bytes()
    assert 2 * half == full
    with pytest.raises(B.IppdError):
        lay.set_option(B.OPT_KERNEL, 1)
    with pytest.raises(B.IppdError):
        lay.set_option(B.OPT_KV_DTYPE, 7)


@pytest.mark.parametrize("tiles_per_split", [0, 3])
def test_one_launch_step_equals_append_then_attention_bit_for_bit_e4m3(tiles_per_split):
    # the fused append writes the same bytes as ippd_append_kv(STEP), and the attention then computes the same bits
    from test_gpu_invariance import _base
    base = _base()
    res = []
    for fused in (False, True):
        run = PoisonedRunner(base, out_dtype=B.F32, tiles_per_split=tiles_per_split, fused=fused, layers_per_call=1,
                             kv_dtype=B.KV_E4M3)
        run.load_header()
        outs = []
        for s in range(base.n_steps):
            act, out = run.run_step(s)
            run.check()
            outs.append(out.clone())
        res.append((outs, run.cache.clone()))
    for a, b in zip(res[0][0], res[1][0]):
        assert torch.equal(a, b)
    assert torch.equal(res[0][1], res[1][1])


def test_question_order_does_not_change_an_answer_e4m3():
    from test_gpu_invariance import Remapped, _all_steps, _base, _close
    base = _base()
    ref = _all_steps(base, kv_dtype=B.KV_E4M3)
    r = np.random.default_rng(9)
    perm = np.concatenate([lo + r.permutation(hi - lo) for lo, hi in zip(base.q_begin[:-1], base.q_begin[1:])])
    got = _all_steps(Remapped.of(base, perm), kv_dtype=B.KV_E4M3)
    for (j, s), o in got.items():
        _close(o, ref[(int(perm[j]), s)], f"permuted question {j} step {s}, e4m3 cache")
