"""Questions are independent of each other (paper Sec. 3: every triplet is its own prompt; Sec. 4.2: finished answers
simply stop being appended): on the CUDA path an answer's output may depend on nothing but its own context, question and
answer tokens.  Checked through the C ABI: question order, duplicated questions, batch composition, questions dropping
out, re-running a step; group sizes 2 and 16, bf16 output, 256-token branch alignment."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from gpu_util import B, W, PoisonedRunner, compare_step, gate, oracle_step  # noqa: E402


class Remapped(W.Workload):
    """Question j of this workload is question src[j] of `base` (same prompt): a permutation reorders the questions of
    a prompt, a repeated entry duplicates one.  Every raw tensor follows its question."""

    @staticmethod
    def of(base, src):
        src = np.asarray(src, dtype=np.int64)
        assert (base.prompt_of[src] == np.sort(base.prompt_of[src])).all()
        q_count = np.bincount(base.prompt_of[src], minlength=base.n_prompts).astype(np.int32)
        wl = Remapped(base.name + "-remapped", base.geom, base.seed, base.ctx_len, q_count, base.q_len[src],
                      base.stop[src], base.max_new[src], int(base.stop[src].max()))
        wl.base, wl.src = base, src
        return wl

    def question_kv(self, k, layer, device="cpu"):
        return self.base.question_kv(int(self.src[k]), layer, device)

    def step_q(self, s, layer, qids, device="cpu"):
        return self.base.step_q(s, layer, self.src[np.asarray(qids, dtype=np.int64)], device)

    def step_kv(self, s, layer, qids, device="cpu"):
        return self.base.step_kv(s, layer, self.src[np.asarray(qids, dtype=np.int64)], device)


def _base():
    geom = W.Geometry(2, 8, 2, 128, 5e5)
    r = np.random.default_rng(3)
    qc = [7, 40, 3]
    nq = sum(qc)
    ql = r.integers(2, 60, nq).tolist()
    ql[8] = 150
    stop = r.integers(2, 6, nq).tolist()
    return W.custom_workload("invariance", geom, 55, [333, 900, 64], qc, ql, stop)


def _all_steps(wl, **kw):
    """Outputs of every step: {(question, step): [layers, Hq, D]} (fp32 output)."""
    run = PoisonedRunner(wl, out_dtype=B.F32, **kw)
    run.load_header()
    res = {}
    for s in range(wl.n_steps):
        act, out = run.run_step(s)
        run.check()
        o = out.cpu().numpy()
        for i, k in enumerate(act):
            res[(int(k), s)] = o[:, i]
    return res


def _close(a, b, what):
    # Two placements of the same row differ only in how its keys were grouped into tiles, i.e. in the reference
    # maxima its probabilities were rounded against: a few 2^-9 of the row's size.
    rms = np.sqrt((b.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
    err = np.abs(a.astype(np.float64) - b) / rms
    assert err.max() <= 1.5e-2 and err.mean() <= 2e-3, f"{what}: {err.max():.3e} {err.mean():.3e}"


def test_question_order_and_duplicates_do_not_change_an_answer():
    base = _base()
    ref = _all_steps(base)
    r = np.random.default_rng(9)
    perm = np.concatenate([lo + r.permutation(hi - lo) for lo, hi in zip(base.q_begin[:-1], base.q_begin[1:])])
    got = _all_steps(Remapped.of(base, perm))
    for (j, s), o in got.items():
        _close(o, ref[(int(perm[j]), s)], f"permuted question {j} step {s}")
    # duplicates: question 8 (the 150-token one) three times in prompt 1, question 0 twice in prompt 0
    src = np.array([0, 0, 1, 2, 3, 4, 5, 6] + [8, 7, 8, 9, 8] + list(range(10, 47)) + [47, 48, 49])
    wl = Remapped.of(base, src)
    got = _all_steps(wl)
    for (j, s), o in got.items():
        _close(o, ref[(int(src[j]), s)], f"duplicated question {j} step {s}")


def test_other_prompts_and_dropped_questions_do_not_change_an_answer():
    base = _base()
    ref = _all_steps(base)
    # batch composition: prompt 1 alone
    lo, hi = int(base.q_begin[1]), int(base.q_begin[2])
    alone = W.custom_workload("alone", base.geom, base.seed, [int(base.ctx_len[1])], [hi - lo], base.q_len[lo:hi].tolist(),
                              base.stop[lo:hi].tolist())

    class Alone(Remapped):
        def ctx_kv(self, b, layer, device="cpu", t0=0, t1=None):
            return self.base.ctx_kv(1, layer, device, t0, t1)

    wl = Alone(alone.name, alone.geom, alone.seed, alone.ctx_len, alone.q_count, alone.q_len, alone.stop, alone.max_new,
               alone.n_steps)
    wl.base, wl.src = base, np.arange(lo, hi)
    got = _all_steps(wl)
    for (j, s), o in got.items():
        _close(o, ref[(lo + j, s)], f"prompt alone, question {j} step {s}")
    # questions dropping out: the same run, but every third question stops after its first step (earlier than its
    # seeded stop); the others' outputs must not move
    early = base.stop.copy()
    early[::3] = 1
    wl2 = W.custom_workload("early", base.geom, base.seed, base.ctx_len.tolist(), base.q_count.tolist(),
                            base.q_len.tolist(), early.tolist(), base.max_new.tolist())
    got = _all_steps(wl2)
    assert len(got) < len(ref)
    for (k, s), o in got.items():
        _close(o, ref[(k, s)], f"with early stops, question {k} step {s}")


@pytest.mark.parametrize("kernel", [1, 2])
def test_rerunning_a_step_is_idempotent(kernel):
    # slot and position derive from (question, answer index) alone: a second run of the same step rewrites the same
    # cache slots with the same bits and returns the same output bit for bit; the next step is unaffected
    base = _base()
    run = PoisonedRunner(base, out_dtype=B.F32, kernel=kernel)
    run.load_header()
    act, first = run.run_step(0)
    snapshot = run.cache.clone()
    act2, second = run.run_step(0)
    run.check()
    assert torch.equal(first, second)
    assert torch.equal(snapshot, run.cache)
    cache = {}
    compare_step(run, 1, [0, 1], range(2), cache, "after a re-run")


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("hq,hkv", [(4, 2), (32, 2)])
def test_group_sizes_2_and_16(kernel, hq, hkv):
    # G = 2: 64 questions fill a 128-row block; G = 16: eight questions do, so 20 questions span three blocks
    nq = 70 if hq == 4 else 20
    r = np.random.default_rng(hq)
    wl = W.custom_workload("g", W.Geometry(1, hq, hkv, 128, 5e5), 13, [400, 10], [nq, 2],
                           r.integers(1, 50, nq + 2).tolist(), r.integers(1, 4, nq + 2).tolist())
    run = PoisonedRunner(wl, out_dtype=B.F32, kernel=kernel)
    run.load_header()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, [0], range(hkv), cache, f"G={hq // hkv}")


@pytest.mark.parametrize("kernel", [1, 2])
def test_bf16_output_and_256_token_branch_alignment(kernel):
    r = np.random.default_rng(21)
    qc = [9, 4]
    ql = r.integers(1, 200, sum(qc)).tolist()
    wl = W.custom_workload("bf16-256", W.Geometry(2, 8, 2, 128, 5e5), 19, [500, 129], qc, ql,
                           r.integers(1, 5, sum(qc)).tolist(), [130] * sum(qc))
    run = PoisonedRunner(wl, out_dtype=B.BF16, kernel=kernel, branch_align=256)
    run.load_header()
    tabs = run.layout.layout_tables()
    assert (tabs["branch_off"] % 256 == 0).all()
    cache = {}
    for s in range(wl.n_steps):
        compare_step(run, s, [0, 1], range(2), cache, "bf16 out, align 256")


@pytest.mark.parametrize("tiles_per_split", [0, 3, 1000])
def test_one_launch_step_equals_append_then_attention_bit_for_bit(tiles_per_split):
    # ippd_decode_step writes the step's K~/V from inside the attention kernel; the cache and the outputs must be the
    # ones ippd_append_kv(STEP) + ippd_decode_attention produce (same tiles, same arithmetic: bitwise), for whole
    # sequences per CTA, for the library's own split and for cuts every three tiles (branch tiles cut from their
    # context, tokens of one branch appended by different CTAs)
    base = _base()
    res = []
    for fused in (False, True):
        run = PoisonedRunner(base, out_dtype=B.F32, tiles_per_split=tiles_per_split, fused=fused, layers_per_call=1)
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
