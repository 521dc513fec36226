"""C-ABI library on the CPU machine: it loads, exports what the header declares, and its host-only
entry points (layout tables, sizes, argument checks) agree bit for bit with the oracle."""
import os
import re

import numpy as np
import pytest

from oracle import ippd_oracle as orc
from paper_2609_05707_b200 import build as ippd_build

ippd_build.build()
from paper_2609_05707_b200 import binding as B  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "ippd.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(ippd_[a-z_]+)\s*\(", hdr)))
    assert "ippd_build_layout" in declared and "ippd_append_kv" in declared and "ippd_decode_attention" in declared
    for name in declared:
        assert hasattr(B.lib, name), name
    assert sorted(B.EXPORTS) == declared


@pytest.mark.parametrize("seed", range(6))
def test_layout_tables_bit_exact_vs_oracle(seed):
    r = np.random.default_rng(seed)
    nb = int(r.integers(1, 6))
    ctx = r.integers(0, 700, nb)
    qc = r.integers(1, 9, nb)
    nq = int(qc.sum())
    ql = r.integers(1, 70, nq)
    mn = r.integers(1, 300, nq)
    align = int(r.choice([128, 256]))
    shared = int([0, 1, 127, 128, 300, 0][seed])  # an instruction shared by all prompts
    lay = B.Layout(B.make_geometry(2, 8, 2, 64, 1e4, branch_align=align), ctx, qc, ql, mn, shared_len=shared)
    got = lay.layout_tables()
    want = orc.layout(ctx, qc, ql, mn, align, B.TILE_TOKENS, shared_len=shared)
    assert got["n_shared_tokens"] == shared and got["n_header_tokens"] == len(want["hdr_pos_virt"])
    for key in ["q_begin", "prompt_of", "branch_off", "ctx_tile_off", "hdr_begin", "hdr_pos_virt", "hdr_ctx_id",
                "hdr_qtn_id"]:
        np.testing.assert_array_equal(got[key], want[key], err_msg=key)
    assert got["n_questions"] == want["n_questions"] and got["n_branch_slots"] == want["branch_off"][-1]
    assert got["n_tiles"] == want["ctx_tile_off"][-1] + want["branch_off"][-1] // B.TILE_TOKENS
    # segments are disjoint, ordered and aligned
    bo = got["branch_off"]
    assert (np.diff(bo) >= ql + mn).all() and (bo % align == 0).all()
    nbytes, al = lay.cache_bytes()
    assert nbytes == 2 * 2 * got["n_tiles"] * 2 * 128 * 64 * 2 and al == 256


def test_host_argument_checks():
    g = B.make_geometry(1, 8, 2, 64, 1e4)
    ok = ([16], [1], [4], [4])
    bad = [
        (B.make_geometry(1, 8, 3, 64, 1e4), *ok),          # Hq % Hkv
        (B.make_geometry(1, 8, 2, 96, 1e4), *ok),          # head_dim
        (B.make_geometry(1, 8, 2, 64, 1e4, branch_align=100), *ok),
        (B.make_geometry(0, 8, 2, 64, 1e4), *ok),
        (g, [-1], [1], [4], [4]),
        (g, [16], [1], [0], [4]),
        (g, [16], [1], [4], [0]),
        (g, [2**31 - 10], [1], [8], [8]),                  # position overflow
    ]
    for args in bad:
        with pytest.raises(B.IppdError) as e:
            B.Layout(*args)
        assert e.value.code == B.ERR_INVALID_ARG
    lay = B.Layout(g, *ok)
    with pytest.raises(B.IppdError) as e:
        lay.begin_step([0], [0])
    assert e.value.code == B.ERR_NOT_BOUND
    with pytest.raises(B.IppdError) as e:
        lay.set_option(99, 1)
    assert e.value.code == B.ERR_INVALID_ARG
    assert lay.workspace_bytes(1) > 0 and lay.step_stage_bytes(1) > 0
    n = lay.export_mask.__self__  # method exists; the sequence-length query is host-only
    import ctypes as C
    cnt = C.c_int64()
    na = np.array([2], dtype=np.int32)
    assert B.lib.ippd_export_mask(lay._h, 0, na.ctypes.data_as(C.POINTER(C.c_int32)), None, C.byref(cnt)) == 0
    assert cnt.value == 16 + 4 + 2


@pytest.mark.parametrize("branch_tokens", [300, 4096, 8192])
def test_step_descriptor_fits_its_staging_slot_for_long_branches(branch_tokens):
    # The per-quarter packing of the branch tiles may cut a full 16-group run into several pieces; the staging slot is
    # sized for that.  Plans the last admissible step of layouts whose branches span many cache tiles (host-only).
    r = np.random.default_rng(branch_tokens)
    for G, hq in [(4, 8), (1, 2), (8, 16)]:
        qc = [32, 5, 70]
        nq = sum(qc)
        ql = r.integers(1, 60, nq)
        mn = np.maximum(1, branch_tokens - ql).astype(np.int32)
        lay = B.Layout(B.make_geometry(2, hq, hq // G, 128, 5e5), [1000, 0, 130], qc, ql, mn)
        for kernel in (1, 2):
            lay.set_option(B.OPT_KERNEL, kernel)
            for tps in (0, 1):
                lay.set_option(B.OPT_TILES_PER_SPLIT, tps)
                act = np.arange(nq, dtype=np.int32)
                for idx in (mn - 1, np.minimum(mn - 1, r.integers(0, branch_tokens, nq))):
                    need, cap = lay.step_descriptor_bytes(act, idx.astype(np.int32))
                    assert 0 < need <= cap, (G, kernel, tps, need, cap)
        # a subset of the questions can only need less
        need_sub, cap = lay.step_descriptor_bytes(act[::3], (mn - 1)[::3])
        assert need_sub <= cap
