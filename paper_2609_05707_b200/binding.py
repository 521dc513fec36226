"""Thin ctypes binding of libippd.so: argument marshalling only, same names as the C ABI.

Every step of the decode path runs inside the CUDA library; there is no Python or
CPU fallback.  Importing this module raises if the library has not been built
(`python -m paper_2609_05707_b200.build`).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libippd.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_05707_b200.build`")
lib = C.CDLL(_LIB_PATH)

OK, ERR_INVALID_ARG, ERR_OOM, ERR_CAPACITY, ERR_NOT_BOUND, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
BF16, F32 = 0, 1
TILE_TOKENS = 128
STATIC_SCRATCH_BYTES = 64 << 20
APPEND_CONTEXT, APPEND_QUESTION, APPEND_STEP, APPEND_SHARED, APPEND_HEADER = 0, 1, 2, 3, 4
OPT_KERNEL, OPT_LAYERS_PER_CALL, OPT_TILES_PER_SPLIT, OPT_WAIT_LIMIT_US, OPT_PROFILE, OPT_KV_DTYPE = 1, 2, 3, 4, 5, 6
KV_BF16, KV_E4M3 = 0, 1

EXPORTS = ["ippd_build_layout", "ippd_build_layout_shared", "ippd_layout_tables", "ippd_cache_bytes", "ippd_bind_cache", "ippd_set_option",
           "ippd_begin_step", "ippd_step_descriptor_bytes", "ippd_append_kv", "ippd_workspace_bytes", "ippd_decode_attention", "ippd_decode_step", "ippd_decode_step_grouped", "ippd_prefill_attention", "ippd_decode_attention_static",
           "ippd_decode_step_host", "ippd_decode_step_host_async", "ippd_host_steps_wait", "ippd_step_stage_bytes", "ippd_export_mask", "ippd_poll_status", "ippd_profile_read", "ippd_read_probe", "ippd_host_time_read",
           "ippd_launch_count", "ippd_last_error", "ippd_destroy_layout"]


class Geometry(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("rope_theta", C.c_double), ("branch_align", C.c_int32),
                ("out_dtype", C.c_int32)]


class Tables(C.Structure):
    _fields_ = [("q_begin", C.POINTER(C.c_int32)), ("prompt_of", C.POINTER(C.c_int32)),
                ("q_len", C.POINTER(C.c_int32)), ("ctx_len", C.POINTER(C.c_int32)),
                ("branch_off", C.POINTER(C.c_int64)), ("ctx_tile_off", C.POINTER(C.c_int32)),
                ("hdr_begin", C.POINTER(C.c_int64)), ("hdr_pos_virt", C.POINTER(C.c_int32)),
                ("hdr_ctx_id", C.POINTER(C.c_int32)), ("hdr_qtn_id", C.POINTER(C.c_int32)),
                ("n_prompts", C.c_int32), ("n_questions", C.c_int32), ("n_header_tokens", C.c_int64),
                ("n_branch_slots", C.c_int64), ("n_tiles", C.c_int64), ("n_shared_tokens", C.c_int32)]


_vp, _i32, _i64, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
_pi32 = C.POINTER(C.c_int32)
lib.ippd_build_layout.argtypes = [C.POINTER(Geometry), _i32, _pi32, _pi32, _pi32, _pi32, C.POINTER(_vp)]
lib.ippd_build_layout_shared.argtypes = [C.POINTER(Geometry), _i32, _i32, _pi32, _pi32, _pi32, _pi32, C.POINTER(_vp)]
lib.ippd_layout_tables.argtypes = [_vp, C.POINTER(Tables)]
lib.ippd_cache_bytes.argtypes = [_vp, C.POINTER(_sz), C.POINTER(_sz)]
lib.ippd_bind_cache.argtypes = [_vp, _vp, _sz, _vp]
lib.ippd_set_option.argtypes = [_vp, _i32, _i64]
lib.ippd_begin_step.argtypes = [_vp, _pi32, _pi32, _i32, _vp]
lib.ippd_step_descriptor_bytes.argtypes = [_vp, _pi32, _pi32, _i32, C.POINTER(_sz), C.POINTER(_sz)]
lib.ippd_append_kv.argtypes = [_vp, _i32, _i32, _i32, _pi32, _i32, _vp, _vp, _vp]
lib.ippd_workspace_bytes.argtypes = [_vp, _i32, C.POINTER(_sz)]
lib.ippd_decode_attention.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp]
lib.ippd_decode_step.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.ippd_prefill_attention.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.ippd_decode_step_grouped.argtypes = [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.ippd_decode_attention_static.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp]
lib.ippd_decode_step_host.argtypes = [_vp, _pi32, _pi32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
lib.ippd_decode_step_host_async.argtypes = [_vp, _pi32, _pi32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]
lib.ippd_host_steps_wait.argtypes = [_vp, _vp]
lib.ippd_step_stage_bytes.argtypes = [_vp, _i32, C.POINTER(_sz)]
lib.ippd_export_mask.argtypes = [_vp, _i32, _pi32, C.POINTER(C.c_uint8), C.POINTER(_i64)]
lib.ippd_poll_status.argtypes = [_vp, _pi32]
lib.ippd_profile_read.argtypes = [_vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                  C.POINTER(_i64)]
lib.ippd_read_probe.argtypes = [_vp, _i32, _i32, _vp]
lib.ippd_host_time_read.argtypes = [_vp, C.POINTER(C.c_double), C.POINTER(_i64)]
lib.ippd_launch_count.argtypes = [_vp]
lib.ippd_launch_count.restype = _i64
lib.ippd_last_error.restype = C.c_char_p
lib.ippd_destroy_layout.argtypes = [_vp]
lib.ippd_destroy_layout.restype = None


class IppdError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed with {code}: {lib.ippd_last_error().decode()}")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise IppdError(code, where)


def _i32arr(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_pi32)


def _dev(t) -> int:
    """Device (or host) address of a torch tensor / int / None."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    assert t.is_contiguous()
    return t.data_ptr()


class Layout:
    """Owns one ippd_layout_t.  Methods mirror the C entry points one to one."""

    def __init__(self, geom: Geometry, ctx_len, q_count, q_len, max_new, shared_len: int = 0):
        self.geom = geom
        self._h = _vp()
        c, qc, ql, mn = _i32arr(ctx_len), _i32arr(q_count), _i32arr(q_len), _i32arr(max_new)
        if len(c) != len(qc) or len(ql) != len(mn) or int(qc.sum()) != len(ql):
            raise ValueError("ragged arrays do not match")
        if shared_len:
            _check(lib.ippd_build_layout_shared(C.byref(geom), int(shared_len), len(c), _p(c), _p(qc), _p(ql), _p(mn),
                                                C.byref(self._h)), "ippd_build_layout_shared")
        else:
            _check(lib.ippd_build_layout(C.byref(geom), len(c), _p(c), _p(qc), _p(ql), _p(mn), C.byref(self._h)),
                   "ippd_build_layout")
        self._keep = None

    def close(self):
        if self._h:
            lib.ippd_destroy_layout(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def layout_tables(self) -> dict:
        t = Tables()
        _check(lib.ippd_layout_tables(self._h, C.byref(t)), "ippd_layout_tables")
        B, NQ, H = t.n_prompts, t.n_questions, t.n_header_tokens
        arr = lambda p, n, dt: np.ctypeslib.as_array(p, shape=(n,)).astype(dt).copy() if n else np.zeros(0, dt)
        return {"q_begin": arr(t.q_begin, B + 1, np.int32), "prompt_of": arr(t.prompt_of, NQ, np.int32),
                "q_len": arr(t.q_len, NQ, np.int32), "ctx_len": arr(t.ctx_len, B, np.int32),
                "branch_off": arr(t.branch_off, NQ + 1, np.int64), "ctx_tile_off": arr(t.ctx_tile_off, B + 1, np.int32),
                "hdr_begin": arr(t.hdr_begin, B + 1, np.int64), "hdr_pos_virt": arr(t.hdr_pos_virt, H, np.int32),
                "hdr_ctx_id": arr(t.hdr_ctx_id, H, np.int32), "hdr_qtn_id": arr(t.hdr_qtn_id, H, np.int32),
                "n_prompts": B, "n_questions": NQ, "n_header_tokens": H, "n_branch_slots": t.n_branch_slots,
                "n_tiles": t.n_tiles, "n_shared_tokens": t.n_shared_tokens}

    def cache_bytes(self):
        b, a = _sz(), _sz()
        _check(lib.ippd_cache_bytes(self._h, C.byref(b), C.byref(a)), "ippd_cache_bytes")
        return b.value, a.value

    def bind_cache(self, cache, stream: int = 0):
        self._keep = cache
        nbytes = cache.numel() * cache.element_size()
        _check(lib.ippd_bind_cache(self._h, _dev(cache), nbytes, stream), "ippd_bind_cache")

    def set_option(self, key: int, value: int):
        _check(lib.ippd_set_option(self._h, key, value), "ippd_set_option")

    def begin_step(self, active_q, answer_idx, stream: int = 0):
        a, s = _i32arr(active_q), _i32arr(answer_idx)
        _check(lib.ippd_begin_step(self._h, _p(a), _p(s), len(a), stream), "ippd_begin_step")

    def step_descriptor_bytes(self, active_q, answer_idx):
        """(bytes of the descriptor begin_step would stage for this step, capacity of a staging slot); host-only."""
        a, s = _i32arr(active_q), _i32arr(answer_idx)
        b, c = _sz(), _sz()
        _check(lib.ippd_step_descriptor_bytes(self._h, _p(a), _p(s), len(a), C.byref(b), C.byref(c)),
               "ippd_step_descriptor_bytes")
        return b.value, c.value

    def append_kv(self, layer_begin: int, layer_count: int, kind: int, ids, k_raw, v_raw, stream: int = 0):
        i = _i32arr(ids if ids is not None else [])
        _check(lib.ippd_append_kv(self._h, layer_begin, layer_count, kind, _p(i) if len(i) else None, len(i),
                                  _dev(k_raw), _dev(v_raw), stream), "ippd_append_kv")

    def workspace_bytes(self, layer_count: int) -> int:
        b = _sz()
        _check(lib.ippd_workspace_bytes(self._h, layer_count, C.byref(b)), "ippd_workspace_bytes")
        return b.value

    def decode_attention(self, layer_begin: int, layer_count: int, q_raw, out, workspace, stream: int = 0):
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_decode_attention(self._h, layer_begin, layer_count, _dev(q_raw), _dev(out), _dev(workspace),
                                         ws_bytes, stream), "ippd_decode_attention")

    def decode_step(self, layer_begin: int, layer_count: int, q_raw, k_raw, v_raw, out, workspace, stream: int = 0):
        """append_kv(STEP) + decode_attention in one launch."""
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_decode_step(self._h, layer_begin, layer_count, _dev(q_raw), _dev(k_raw), _dev(v_raw), _dev(out),
                                    _dev(workspace), ws_bytes, stream), "ippd_decode_step")

    def prefill_attention(self, layer_begin: int, layer_count: int, q_raw, k_raw, v_raw, out, workspace,
                          stream: int = 0):
        """Prefill of the stacked header: appends its K/V and returns the attention output of every header token."""
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_prefill_attention(self._h, layer_begin, layer_count, _dev(q_raw), _dev(k_raw), _dev(v_raw),
                                          _dev(out), _dev(workspace), ws_bytes, stream), "ippd_prefill_attention")

    def decode_step_grouped(self, layers_per_call: int, q_raw, k_raw, v_raw, out, workspace, stream: int = 0):
        """decode_step for all layers of the step, `layers_per_call` layers per launch."""
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_decode_step_grouped(self._h, layers_per_call, _dev(q_raw), _dev(k_raw), _dev(v_raw), _dev(out),
                                            _dev(workspace), ws_bytes, stream), "ippd_decode_step_grouped")

    def decode_attention_static(self, layer_begin: int, layer_count: int, q_raw, out, stream: int = 0):
        """Same result as decode_attention, for callers that may not allocate: the split-KV scratch is the
        library's built-in device array (STATIC_SCRATCH_BYTES per GPU) instead of a caller workspace."""
        _check(lib.ippd_decode_attention_static(self._h, layer_begin, layer_count, _dev(q_raw), _dev(out), stream),
               "ippd_decode_attention_static")

    def step_stage_bytes(self, n_active: int) -> int:
        b = _sz()
        _check(lib.ippd_step_stage_bytes(self._h, n_active, C.byref(b)), "ippd_step_stage_bytes")
        return b.value

    def decode_step_host(self, active_q, answer_idx, host_q, host_k, host_v, host_out, dev_stage, workspace,
                         stream: int = 0):
        a, s = _i32arr(active_q), _i32arr(answer_idx)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_decode_step_host(self._h, _p(a), _p(s), len(a), _dev(host_q), _dev(host_k), _dev(host_v),
                                         _dev(host_out), _dev(dev_stage), dev_stage.numel() * dev_stage.element_size(),
                                         _dev(workspace), ws_bytes, stream), "ippd_decode_step_host")

    def decode_step_host_async(self, active_q, answer_idx, host_q, host_k, host_v, host_out, dev_stage, workspace,
                               stream: int = 0):
        a, s = _i32arr(active_q), _i32arr(answer_idx)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib.ippd_decode_step_host_async(self._h, _p(a), _p(s), len(a), _dev(host_q), _dev(host_k),
                                               _dev(host_v), _dev(host_out), _dev(dev_stage),
                                               dev_stage.numel() * dev_stage.element_size(), _dev(workspace), ws_bytes,
                                               stream), "ippd_decode_step_host_async")

    def host_steps_wait(self, stream: int = 0):
        _check(lib.ippd_host_steps_wait(self._h, stream), "ippd_host_steps_wait")

    def export_mask(self, prompt: int, n_answer) -> np.ndarray:
        na = _i32arr(n_answer)
        n = _i64()
        _check(lib.ippd_export_mask(self._h, prompt, _p(na), None, C.byref(n)), "ippd_export_mask")
        out = np.zeros((n.value, n.value), dtype=np.uint8)
        _check(lib.ippd_export_mask(self._h, prompt, _p(na), out.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(n)),
               "ippd_export_mask")
        return out

    def poll_status(self) -> int:
        w = _i32()
        _check(lib.ippd_poll_status(self._h, C.byref(w)), "ippd_poll_status")
        return w.value

    def profile_read(self) -> dict:
        a, m, p, n = C.c_double(), C.c_double(), C.c_double(), _i64()
        _check(lib.ippd_profile_read(self._h, C.byref(a), C.byref(m), C.byref(p), C.byref(n)), "ippd_profile_read")
        return {"attention_ms": a.value, "merge_ms": m.value, "append_ms": p.value, "n_attention": n.value}

    def read_probe(self, layer_begin: int, layer_count: int, stream: int = 0):
        _check(lib.ippd_read_probe(self._h, layer_begin, layer_count, stream), "ippd_read_probe")

    def host_time_read(self) -> dict:
        us, n = C.c_double(), _i64()
        _check(lib.ippd_host_time_read(self._h, C.byref(us), C.byref(n)), "ippd_host_time_read")
        return {"begin_step_us": us.value, "steps": n.value}

    def launch_count(self) -> int:
        return int(lib.ippd_launch_count(self._h))


def make_geometry(n_layers, n_q_heads, n_kv_heads, head_dim, rope_theta, branch_align=TILE_TOKENS,
                  out_dtype=BF16) -> Geometry:
    return Geometry(n_layers, n_q_heads, n_kv_heads, head_dim, float(rope_theta), branch_align, out_dtype)
