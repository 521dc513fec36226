"""The seeded input generator: determinism, CPU reference hash, distribution, config shapes."""
import numpy as np
import torch

from paper_2609_05707_b200 import workloads as W


def test_tensor_hash_equals_python_int_hash():
    xs = [0, 1, 2**40 + 12345, 2**63 - 1, -1, -(2**62)]
    got = W.mix64(torch.tensor(xs, dtype=torch.int64))
    for x, g in zip(xs, got.tolist()):
        assert g & ((1 << 64) - 1) == W.mix64_int(x)


def test_values_are_deterministic_slices_and_unit_normal():
    a = W.values(5, W.stream_id(W.K_CTX, 3), 0, 1 << 20)
    b = W.values(5, W.stream_id(W.K_CTX, 3), 1000, 500)
    assert a.dtype == torch.bfloat16
    assert torch.equal(a[1000:1500], b)
    c = W.values(5, W.stream_id(W.V_CTX, 3), 0, 1 << 20)
    assert not torch.equal(a, c)
    f = a.double()
    assert abs(f.mean().item()) < 5e-3 and abs(f.var().item() - 1.0) < 1e-2
    assert abs((f * c.double()).mean().item()) < 5e-3
    # quantile table is antisymmetric and monotone
    t = W.normal_table().double()
    assert torch.equal(t, -t.flip(0)) and (t[1:] >= t[:-1]).all()


def test_config_shapes_follow_the_recipe():
    c1 = W.make_workload("C1")
    assert (c1.geom.n_q_heads, c1.geom.n_kv_heads, c1.geom.head_dim) == (8, 2, 64)
    assert list(c1.ctx_len) == [512] and c1.n_questions == 4 and c1.n_steps == 32
    assert c1.q_len.min() >= 8 and c1.q_len.max() <= 24 and c1.question_tokens() == 128
    c2 = W.make_workload("C2")
    assert c2.n_questions == 16 and c2.q_len.min() >= 16 and c2.q_len.max() <= 48 and c2.question_tokens() == 2048
    c3 = W.make_workload("C3")
    assert c3.stop.min() >= 8 and c3.stop.max() <= 256 and c3.n_steps == c3.stop.max()
    assert len(c3.active(int(c3.stop.min()))) < 32
    c4 = W.make_workload("C4")
    assert c4.n_prompts == 32 and c4.ctx_len.min() >= 1024 and c4.ctx_len.max() <= 4096
    assert c4.q_count.min() >= 4 and c4.q_count.max() <= 64 and c4.n_questions == c4.q_count.sum()
    c5 = W.make_workload("C5")
    assert c5.geom.n_layers == 80 and c5.n_questions == 1024 and c5.stop.max() <= 64
    s1, s2 = W.make_workload("S1"), W.make_workload("S2")
    for wl, (Lr, Qr, nr, sr) in ((s1, ((2600, 4400), (22, 38), (8, 16), (6, 40))),
                                 (s2, ((170, 280), (6, 12), (9, 17), (4, 30)))):
        assert wl.n_prompts == 6 and wl.geom.n_layers == 32 and wl.geom.head_dim == 128
        assert Lr[0] <= wl.ctx_len.min() and wl.ctx_len.max() <= Lr[1]
        assert Qr[0] <= wl.q_count.min() and wl.q_count.max() <= Qr[1]
        assert nr[0] <= wl.q_len.min() and wl.q_len.max() <= nr[1]
        assert sr[0] <= wl.stop.min() and wl.stop.max() <= sr[1] and wl.n_steps == wl.stop.max()
    # layer override keeps the values of the layers that remain
    a = W.make_workload("C2", n_layers=2).ctx_kv(0, 1, t0=5, t1=9)[0]
    b = c2.ctx_kv(0, 1, t0=5, t1=9)[0]
    assert torch.equal(a, b)
    sb = c2.step_bytes(0)
    assert sb["context"] == 2048 * 4096 * 32 and sb["branch"] == int((c2.q_len + 1).sum()) * 4096 * 32


def test_sweep_and_shared_workloads_follow_their_recipes():
    wl = W.make_workload("SWEEP-L8192-Q4")
    assert wl.ctx_len.tolist() == [8192] and wl.q_count.tolist() == [4] and wl.q_len.tolist() == [32] * 4
    assert wl.n_steps == 16 and (wl.stop == 16).all() and wl.geom.n_layers == 32
    assert W.make_workload("SWEEP-L2048-Q32", n_layers=2).geom.n_layers == 2
    s3 = W.make_workload("S3")
    assert s3.shared_len == 2754 and s3.n_prompts == 12
    assert (s3.ctx_len >= 550).all() and (s3.ctx_len <= 920).all() and (s3.stop >= 1).all() and (s3.stop <= 11).all()
    k, v = s3.shared_kv(3)
    assert k.shape == (2754, 8, 128) and not torch.equal(k, v)
    # the instruction is counted once per step in the algorithmic bytes, every context once
    b = s3.step_bytes(0)
    assert b["context"] == (2754 + int(s3.ctx_len.sum())) * s3.geom.kv_bytes_per_token * 32


def test_step_bytes_count_the_cache_by_its_element_size():
    # algorithmic bytes of a step: the cache part halves on the 8-bit cache, queries and outputs stay bf16
    wl = W.make_workload("C2")
    g = wl.geom
    for s in (0, 63, 127):
        b2, b1 = wl.step_bytes(s), wl.step_bytes(s, 1)
        assert b1["context"] * 2 == b2["context"] and b1["branch"] * 2 == b2["branch"]
        assert b1["q_out"] == b2["q_out"] == len(wl.active(s)) * g.n_q_heads * g.head_dim * 2 * 2 * g.n_layers
        assert b1["total"] == b1["context"] + b1["branch"] + b1["q_out"]
        # by hand: one context of 2048 tokens, 16 branches of n_k + s + 1 tokens, K and V, 8 KV heads x 128 dims x 2 bytes
        tokens = 2048 + int((wl.q_len[wl.active(s)] + s + 1).sum())
        assert b2["context"] + b2["branch"] == tokens * 2 * g.n_kv_heads * g.head_dim * 2 * g.n_layers
