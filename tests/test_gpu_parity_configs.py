"""GPU-vs-oracle parity on every configuration the benchmark names, through the C ABI.

* prompt passes of more than one block of 1024 rows (later blocks attend over earlier ones,
  ragged last block): next-token logits on top of the cache they leave, against the oracle;
* the Llama-2-13B and Llama-3-8B shapes (two-layer models: the oracle finishes in seconds):
  teacher-forced exit and final logits, passes of 16 + 9 and 16 + 5 rows; their projection
  shapes and the 128256-row LM head on sampled output rows;
* the Llama-2-7B shape at full depth on 17 teacher-forced positions (a 16-row and a 1-row pass);
* per-step accepted counts of the self-speculative loop against the oracle (Appendix A.4's
  `match`), early-exit generation (Sec. 4.2) and the "without exit-cache reuse" ablation
  (Sec. 4.3.3, Table 7) against the oracle's routines.

Tolerances: logits max|delta| <= 3e-2 * max|logit| (tests/helpers.py); integer results are
compared exactly wherever the oracle's decision is clear of that tolerance.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import ls_oracle as O
from paper_2404_16710_b200 import binding as B
from paper_2404_16710_b200 import synth
from tests.helpers import LOGIT_TOL, assert_logits_close, bits, make_pair, vals

pytestmark = pytest.mark.gpu
PATHS = [B.LS_LINEAR_FMA, B.LS_LINEAR_MMA]
TINY = synth.WORKLOADS["tiny"]
ODD_G2 = synth.Shape("odd-g2", 3, 104, 6, 3, 64, 200, 301)


def two_layers(shape, name):
    return replace(shape, name=name, n_layers=2)


def rel_margins(z):
    """top-1 minus top-2 of every row, relative to the largest |logit| of the whole array"""
    part = np.partition(z, -2, axis=1)
    return (part[:, -1] - part[:, -2]) / np.abs(z).max()


# ------------------------------------------------------------------ prompt pass of several blocks
LONG_PROMPTS = [(TINY.shape, 1025, None), (TINY.shape, 2100, None), (TINY.shape, 3001, None),
                (ODD_G2, 1100, 6.0), (ODD_G2, 2100, 6.0), (two_layers(synth.LLAMA2_7B, "7b-2-layers"), 1100, None),
                # head dim 128: the second block (299 rows at position 1024) also runs the tcgen05 attention kernel,
                # over the first block's cache; the 8B shape with four query heads per KV head
                (two_layers(synth.LLAMA2_7B, "7b-2-layers"), 1324, None),
                (two_layers(synth.LLAMA3_8B, "8b-2-layers"), 1324, None)]


@pytest.mark.parametrize("shape,n_prompt,amp", LONG_PROMPTS, ids=lambda v: getattr(v, "name", str(v)))
def test_prompt_pass_of_several_blocks_gives_the_oracle_logits(shape, n_prompt, amp):
    """A prompt of more than 1024 rows goes through the layers block by block: the rows of a
    later block are rotated and cached at positions >= 1024 and attend over the earlier blocks'
    cache.  The next-token logits on top of that cache are compared with the oracle's
    teacher-forced final logits at the last prompt position (every cached k, v of every layer
    enters them)."""
    gm, om = make_pair(shape, 5, 1, 0.3, n_prompt + 16, page_size=64, max_draft=4, amplify=amp)
    prompt = synth.make_prompt(shape.vocab, n_prompt, 12)
    B.ls_prefill(gm.h, prompt)
    got = B.ls_debug_next_logits(gm.h, shape.vocab)
    _, ref = om.teacher_logits_tail(prompt, 1, n_prompt - 1, want_exit=False)
    r = assert_logits_close(got, ref[0], "next-token logits after a prompt pass of several blocks")
    # the loops that start from this cache agree with each other bit for bit ...
    full = gm.generate_full(prompt, 6)
    spec, _ = gm.generate(prompt, 1, 3, 6)
    np.testing.assert_array_equal(spec, full)
    # ... and their first token is the oracle's wherever its margin allows
    if rel_margins(ref)[0] > LOGIT_TOL:
        assert full[0] == int(ref[0].argmax())
    print(f"{shape.name} prompt {n_prompt}: max|delta|/max|logit| {r:.2e}")


# ------------------------------------------------------------------ 13B and Llama-3-8B shapes
@pytest.mark.parametrize("shape,E,n_ids", [(two_layers(synth.LLAMA2_13B, "13b-2-layers"), 1, 25),
                                           (two_layers(synth.LLAMA3_8B, "8b-2-layers"), 1, 21)],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_teacher_forced_logits_13b_and_8b_shapes(shape, E, n_ids):
    """Passes of 16 + 9 rows (13B shape: D 5120, 40 heads, F 13824) and 16 + 5 rows (8B shape:
    32/8 grouped heads, F 14336, 128256 logits per row) through the kernels these (N, K) select,
    against the oracle's exit and final logits."""
    gm, om = make_pair(shape, 1234, E, 0.05, 64, max_draft=8)
    ids = synth.make_prompt(shape.vocab, n_ids, 21)
    gex, gfi = gm.debug_logits(ids, E)
    oex, ofi = om.teacher_logits(ids, E)
    r1 = assert_logits_close(gex, oex, "exit logits")
    r2 = assert_logits_close(gfi, ofi, "final logits")
    for g, o in ((gex, oex), (gfi, ofi)):
        safe = rel_margins(o) > LOGIT_TOL
        assert (g.argmax(1)[safe] == o.argmax(1)[safe]).all()
    print(f"{shape.name}: max|delta|/max|logit| exit {r1:.2e} final {r2:.2e}")


def sampled_rows(N, seed):
    return np.unique(np.concatenate([[0, 15, 16, N - 17, N - 1], np.random.default_rng(seed).integers(0, N, 40)]))


def rnd(shape, seed, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return torch.randn(shape, generator=g, device="cuda") * scale


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("N,K", [(5120, 13824), (15360, 5120), (5120, 5120), (6144, 4096)])
@pytest.mark.parametrize("M", [1, 5, 9, 13])
def test_linear_13b_and_8b_shapes_sampled_rows(path, N, K, M):
    """down-proj, q|k|v and o-proj of the 13B shape, q|k|v of the 8B shape."""
    w = rnd((N, K), 77, 0.05).bfloat16()
    h = rnd((M, K), 78).bfloat16()
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    B.ls_op_linear(path, w, h, out)
    torch.cuda.synchronize()
    rows = sampled_rows(N, 0)
    wb, hv = bits(w[torch.from_numpy(rows).cuda()]), vals(h)
    got = out.cpu().numpy().astype(np.float64)[:, rows]
    for m in range(M):
        ref = O.linear(wb, hv[m])
        np.testing.assert_allclose(got[m], ref, rtol=0, atol=1e-5 * np.abs(ref).max())


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("F,K", [(13824, 5120), (14336, 4096)])
@pytest.mark.parametrize("M", [1, 5, 9, 13])
def test_gate_up_swiglu_13b_and_8b_shapes_sampled_columns(path, F, K, M):
    wg, wu = rnd((F, K), 20, 0.05).bfloat16(), rnd((F, K), 21, 0.05).bfloat16()
    h = rnd((M, K), 22).bfloat16()
    out = torch.empty((M, F), dtype=torch.bfloat16, device="cuda")
    B.ls_op_gate_up_swiglu(path, wg, wu, h, out)
    torch.cuda.synchronize()
    cols = sampled_rows(F, 1)
    idx = torch.from_numpy(cols).cuda()
    gb, ub, hv = bits(wg[idx]), bits(wu[idx]), vals(h)
    for m in range(M):
        g, u = O.linear(gb, hv[m]), O.linear(ub, hv[m])
        ref = np.array([O.silu(a) for a in g]) * u
        got = vals(out[m])[cols]
        tol = 2.0 ** -8 * np.abs(ref) + 1e-6 * np.abs(ref).max()
        assert (np.abs(got - ref) <= tol).all(), f"row {m}"


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M", [1, 5, 9, 13])
def test_lm_head_argmax_llama3_vocabulary(path, M):
    """128256 logits per row (8016 tiles of 16 rows): the id is the argmax of the kernel's own
    fp32 logits (lowest index on ties), the logits of sampled rows are the oracle's, and the id
    is the oracle's whenever the margin (taken from the kernel's logits, which the sampled rows
    tie to the oracle) is beyond fp32 accumulation error."""
    V, K = 128256, 4096
    w = rnd((V, K), 30, 0.05).bfloat16()
    h = rnd((M, K), 31).bfloat16()
    scratch = torch.empty(B.ls_op_lm_head_scratch_bytes(V), dtype=torch.uint8, device="cuda")
    tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
    B.ls_op_lm_head_argmax(path, w, h, scratch, tok, logits)
    tok2 = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    B.ls_op_lm_head_argmax(path, w, h, scratch, tok2, None)
    torch.cuda.synchronize()
    assert torch.equal(tok, tok2)
    lg = logits.cpu().numpy()
    hv = vals(h)
    for m in range(M):
        assert int(tok[m]) == int(np.argmax(lg[m]))
        top2 = np.argsort(lg[m])[-2:]
        rows = np.unique(np.concatenate([sampled_rows(V, m), top2]))
        ref = O.linear(bits(w[torch.from_numpy(rows).cuda()]), hv[m])
        np.testing.assert_allclose(lg[m][rows].astype(np.float64), ref, rtol=0, atol=1e-5 * np.abs(lg[m]).max())


# ------------------------------------------------------------------ accepted drafts per step
def clear_steps_equal(gm, om, prompt, E, d, ids, acc):
    """Every step of a GPU run against the oracle's exit and final logits, teacher-forced on the
    GPU's own ids.  A step that starts after e emitted tokens accepts n = the number of leading
    i < d with argmax g(x_E) == argmax g(x_L) at generated position e + i (the drafts before a
    mismatch follow the true sequence, the ones after it cannot count).  A step is compared when
    every row it decides on is clear: both margins further from zero than the two sides can
    differ, i.e. 2 * the largest |GPU - oracle| logit difference measured on the same rows.
    -> (steps compared, steps, fraction of clear rows)"""
    P = len(prompt)
    seq = np.concatenate([prompt, ids])
    oex, ofi = om.teacher_logits_tail(seq, E, P - 1)
    gex, gfi = gm.debug_logits(seq, E)
    gex, gfi = gex[P - 1:], gfi[P - 1:]
    assert_logits_close(gex, oex, "exit logits")
    assert_logits_close(gfi, ofi, "final logits")
    tol_e = 2 * np.abs(gex - oex).max() / np.abs(oex).max()
    tol_f = 2 * np.abs(gfi - ofi).max() / np.abs(ofi).max()
    clear = (rel_margins(oex) > tol_e) & (rel_margins(ofi) > tol_f)
    dr, fu = oex.argmax(1), ofi.argmax(1)
    e = checked = 0
    for n_gpu in acc:
        n_ref, ok = 0, True
        for i in range(d):
            if e + i >= len(ids):  # rows past the requested length: the GPU still ran them, the oracle has no ids
                ok = False
                break
            ok = ok and clear[e + i]
            if not ok or dr[e + i] != fu[e + i]:
                break
            n_ref += 1
        if ok and e + n_ref < len(ids) and clear[e + n_ref]:
            assert fu[e + n_ref] == ids[e + n_ref]
            assert n_gpu == n_ref, f"step starting after {e} tokens: accepted {n_gpu}, oracle {n_ref}"
            checked += 1
        e += n_gpu + 1
    print(f"margin tolerances (relative to max|logit|): exit {tol_e:.2e} final {tol_f:.2e}; "
          f"{clear.mean():.2f} of the rows clear")
    return checked, len(acc), float(clear.mean())


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("amp,d,prompt_seed", [(None, 3, TINY.prompt_seed), (None, 5, 7), (None, 8, 9)])
def test_accepted_per_step_equals_the_oracle_on_every_clear_step(path, amp, d, prompt_seed):
    E = TINY.exit_layer
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 160, linear_path=path, amplify=amp)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, prompt_seed)
    ids, acc = gm.generate(prompt, E, d, TINY.max_new)
    np.testing.assert_array_equal(ids, gm.generate_full(prompt, TINY.max_new))
    checked, steps, frac = clear_steps_equal(gm, om, prompt, E, d, ids, acc)
    print(f"path {path} amplify {amp} d {d}: {checked} of {steps} steps clear and equal, accepted/step {acc.mean():.2f}")
    # a step decides on 1 .. d + 1 rows, all of which have to be clear
    assert checked >= steps // 4


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("prompt_seed", [141, 87])
def test_accepted_per_step_equals_the_oracle_run_on_the_safe_prefix(path, prompt_seed):
    """Free-running against the oracle's own self-speculative run: ids and accepted counts are
    equal for every step that ends before the first generated position whose oracle margin --
    of the final OR of the exit logits along the oracle's ids -- is inside the logit tolerance.
    The two prompts were picked (with the oracle alone) for a prefix of 14 tokens."""
    E, d, new = TINY.exit_layer, TINY.num_draft, 40
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 128, linear_path=path, draw_on="cpu")
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, prompt_seed)
    ref_ids, ref_acc, _ = om.generate_spec(prompt, E, d, new)
    oex, ofi = om.teacher_logits_tail(np.concatenate([prompt, ref_ids]), E, len(prompt) - 1)
    low = np.nonzero((rel_margins(oex)[:-1] <= LOGIT_TOL) | (rel_margins(ofi)[:-1] <= LOGIT_TOL))[0]
    k = int(low[0]) if low.size else new
    assert k >= 12, "the prompt no longer gives a long safe prefix: the input recipe changed"
    ids, acc = gm.generate(prompt, E, d, new)
    np.testing.assert_array_equal(ids[:k], ref_ids[:k])
    e = compared = 0
    for s, n in enumerate(ref_acc):
        if e + d >= k:  # the step's rows reach the first low-margin position
            break
        assert acc[s] == n, f"step {s}: accepted {acc[s]}, oracle {n}"
        compared += 1
        e += n + 1
    assert compared >= 3
    print(f"path {path} prompt seed {prompt_seed}: safe prefix {k}, {compared} steps equal: {ref_acc[:compared]}")


# ------------------------------------------------------------------ early exit, no exit-cache reuse
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("amp,prompt_seed", [(None, 87), (None, TINY.prompt_seed), (6.0, 112)])
def test_early_exit_generation_follows_the_oracle(path, amp, prompt_seed):
    """ls_generate_early (Sec. 4.2: every token is argmax g(x_E); its prompt pass runs E layers
    only) against lso_generate_early: equal ids up to the first position whose oracle EXIT-logit
    margin is inside the tolerance, and beyond that every GPU token is the oracle's argmax given
    the GPU's own history wherever that margin is clear."""
    E, new = TINY.exit_layer, 48
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 128, linear_path=path, amplify=amp,
                       draw_on="cpu")
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, prompt_seed)
    P = len(prompt)
    ref = om.generate_early(prompt, E, new)
    ids = gm.generate_early(prompt, E, new)
    assert len(ids) == new
    oex, _ = om.teacher_logits_tail(np.concatenate([prompt, ref]), E, P - 1, want_final=False)
    low = np.nonzero(rel_margins(oex)[:-1] <= LOGIT_TOL)[0]
    k = int(low[0]) if low.size else new
    np.testing.assert_array_equal(ids[:k], ref[:k])
    own, _ = om.teacher_logits_tail(np.concatenate([prompt, ids]), E, P - 1, want_final=False)
    clear = rel_margins(own)[:-1] > LOGIT_TOL
    assert (own.argmax(1)[:-1][clear] == ids[clear]).all()
    print(f"path {path} amplify {amp} seed {prompt_seed}: safe prefix {k}, {int(clear.sum())} of {new} positions clear")
    assert clear.sum() >= new // 5
    if amp is None and prompt_seed == 87:
        assert k >= 12


def test_early_exit_generation_equals_the_golden_ids():
    import json
    import os
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "tiny_workload.json")))
    if "early_exit_ids" not in gold:
        pytest.skip("golden file holds no early-exit ids")
    gm, om = make_pair(TINY.shape, TINY.weight_seed, TINY.exit_layer, TINY.late_scale, 128)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    ref = np.asarray(gold["early_exit_ids"], dtype=np.int32)
    ids = gm.generate_early(prompt, TINY.exit_layer, len(ref))
    oex, _ = om.teacher_logits_tail(np.concatenate([prompt, ref]), TINY.exit_layer, len(prompt) - 1, want_final=False)
    low = np.nonzero(rel_margins(oex)[:-1] <= LOGIT_TOL)[0]
    k = int(low[0]) if low.size else len(ref)
    np.testing.assert_array_equal(ids[:k], ref[:k])


@pytest.mark.parametrize("path", PATHS)
def test_without_exit_cache_reuse_against_the_oracle(path):
    """The "without KVQ reuse" ablation (Sec. 4.3.3, Table 7) recomputes the early layers of the
    d + 1 verify rows; its tokens and accepted counts are those of the method itself, so the
    oracle's lso_generate_spec is the reference: accepted-per-step exactly at zero late scale,
    ids on the safe prefix, every clear step otherwise."""
    E, d = 2, 3
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, 0.0, 128, linear_path=path)
    prompt = synth.make_prompt(TINY.shape.vocab, 10, TINY.prompt_seed)
    B.ls_prefill(gm.h, prompt)
    B.ls_decode_flags(gm.h, E, d, 22, B.LS_DECODE_NO_EXIT_CACHE)
    ids, acc = B.ls_read_output(gm.h, 22)
    oids, oacc, _ = om.generate_spec(prompt, E, d, 22)
    np.testing.assert_array_equal(acc, oacc)
    assert (acc == d).all()
    _, margins, maxabs = om.generate_full(prompt, 22)
    low = np.nonzero(margins <= LOGIT_TOL * maxabs)[0]
    k = int(low[0]) if low.size else 22
    np.testing.assert_array_equal(ids[:k], oids[:k])

    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 160, linear_path=path)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, 87)
    B.ls_prefill(gm.h, prompt)
    B.ls_decode_flags(gm.h, E, d, TINY.max_new, B.LS_DECODE_NO_EXIT_CACHE)
    ids, acc = B.ls_read_output(gm.h, TINY.max_new)
    checked, steps, _ = clear_steps_equal(gm, om, prompt, E, d, ids, acc)
    oids, oacc, _ = om.generate_spec(prompt, E, d, TINY.max_new)
    _, margins, maxabs = om.generate_full(prompt, TINY.max_new)
    low = np.nonzero(margins <= LOGIT_TOL * maxabs)[0]
    k = int(low[0]) if low.size else TINY.max_new
    np.testing.assert_array_equal(ids[:k], oids[:k])
    print(f"path {path}: {checked} of {steps} steps clear and equal, safe prefix {k}")
    assert checked >= steps // 4
