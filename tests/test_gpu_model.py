"""Parity of the whole decode path (through the C ABI) against the CPU oracle, and the
properties that hold at any size.

* teacher-forced exit-layer and final logits: max|delta| <= 3e-2 * max|logit|
  (bf16 weights / activations / KV, fp32 accumulation, against the fp64 oracle);
* free-running ids equal the oracle's up to the first position whose oracle top-1/top-2
  margin is inside that tolerance;
* ls_generate == ls_generate_full bit-exactly for every (E, d) -- the losslessness of
  self-speculative decoding (Sec. 4.3 of the paper), which on the GPU also needs every
  kernel to be independent of the pass size;
* accepted-per-step bookkeeping invariants, the zero-scale case, EOS, a shuffled page
  table, determinism, and the error codes of the boundary.
"""
import numpy as np
import pytest
import torch

from paper_2404_16710_b200 import binding as B
from paper_2404_16710_b200 import synth
from tests.helpers import LOGIT_TOL, assert_logits_close, first_low_margin, make_pair

pytestmark = pytest.mark.gpu
PATHS = [B.LS_LINEAR_FMA, B.LS_LINEAR_MMA]
TINY = synth.WORKLOADS["tiny"]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("E", [1, 2, 4])
def test_teacher_forced_logits_tiny(path, E):
    gm, om = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, linear_path=path)
    ids = synth.make_prompt(TINY.shape.vocab, 41, 99)  # 16 + 16 + 9 rows: full tiles and a ragged tail
    gex, gfi = gm.debug_logits(ids, E)
    oex, ofi = om.teacher_logits(ids, E)
    r1 = assert_logits_close(gex, oex, "exit logits")
    r2 = assert_logits_close(gfi, ofi, "final logits")
    print(f"path {path} E {E}: max|delta|/max|logit| exit {r1:.2e} final {r2:.2e}")
    if E == 4:
        assert np.array_equal(gex, gfi)
    # argmax agrees wherever the oracle's margin is beyond the tolerance
    for g, o in ((gex, oex), (gfi, ofi)):
        part = np.partition(o, -2, axis=1)
        safe = (part[:, -1] - part[:, -2]) > LOGIT_TOL * np.abs(o).max()
        assert (g.argmax(1)[safe] == o.argmax(1)[safe]).all()


@pytest.mark.parametrize("path", PATHS)
def test_teacher_forced_logits_grouped_kv_ragged_shapes(path):
    shape = synth.GPU_MICRO
    gm, om = make_pair(shape, 5, 0, 1.0, 96, page_size=16, linear_path=path, amplify=6.0)
    ids = synth.make_prompt(shape.vocab, 37, 3)
    gex, gfi = gm.debug_logits(ids, 1)
    oex, ofi = om.teacher_logits(ids, 1)
    assert np.abs(ofi).max() > 0.5
    assert_logits_close(gex, oex, "exit logits")
    assert_logits_close(gfi, ofi, "final logits")


@pytest.mark.parametrize("path", PATHS)
def test_free_running_ids_follow_the_oracle_while_margins_allow(path):
    gm, om = make_pair(TINY.shape, TINY.weight_seed, TINY.exit_layer, TINY.late_scale, 128, linear_path=path)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    ref, margins, maxabs = om.generate_full(prompt, TINY.max_new)
    ids = gm.generate_full(prompt, TINY.max_new)
    assert len(ids) == TINY.max_new
    k = first_low_margin(margins, maxabs)
    assert k >= 1
    np.testing.assert_array_equal(ids[:k], ref[:k])
    assert len(gm.generate_early(prompt, 2, 8)) == 8


@pytest.mark.parametrize("path", PATHS)
def test_generate_equals_generate_full_for_every_exit_and_draft(path):
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, TINY.exit_layer, TINY.late_scale, 160, max_draft=15,
                      linear_path=path, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    full = gm.generate_full(prompt, TINY.max_new)
    again = gm.generate_full(prompt, TINY.max_new)
    np.testing.assert_array_equal(full, again)  # deterministic
    for E in (1, 2, 3):
        for d in (1, 2, 3, 5, 8, 15):
            ids, acc = gm.generate(prompt, E, d, TINY.max_new)
            np.testing.assert_array_equal(ids, full, err_msg=f"E={E} d={d}")
            assert ((0 <= acc) & (acc <= d)).all()
            emitted = np.cumsum(acc + 1)
            assert emitted[-1] >= TINY.max_new and (len(emitted) == 1 or emitted[-2] < TINY.max_new)
            st = gm.stats()
            assert st.n_generated == TINY.max_new and st.n_steps == len(acc) and st.n_accepted == acc.sum()
            assert st.host_syncs <= 8 < TINY.max_new  # no host sync per token


@pytest.mark.parametrize("path", PATHS)
def test_zero_late_scale_accepts_every_draft(path):
    E, d = 2, 3
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, 0.0, 128, linear_path=path)
    prompt = synth.make_prompt(TINY.shape.vocab, 10, TINY.prompt_seed)
    ids, acc = gm.generate(prompt, E, d, 22)
    assert (acc == d).all() and len(acc) == -(-22 // (d + 1))
    np.testing.assert_array_equal(ids, gm.generate_full(prompt, 22))
    np.testing.assert_array_equal(ids, gm.generate_early(prompt, E, 22))
    _, oacc, _ = om.generate_spec(prompt, E, d, 22)
    np.testing.assert_array_equal(acc, oacc)


def test_shuffled_page_table_changes_nothing():
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, page_size=16, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, 40, 8)
    a_ids, a_acc = gm.generate(prompt, 2, 3, 48)
    table = np.random.default_rng(0).permutation(128 // 16).astype(np.int32)
    B.ls_set_page_table(gm.h, table)
    b_ids, b_acc = gm.generate(prompt, 2, 3, 48)
    np.testing.assert_array_equal(a_ids, b_ids)
    np.testing.assert_array_equal(a_acc, b_acc)
    with pytest.raises(B.LsError):
        B.ls_set_page_table(gm.h, np.zeros(8, np.int32))  # not a permutation


def test_eos_stops_both_loops_at_the_same_token():
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, oracle=False)
    full = gm.generate_full(prompt, 40)
    eos = int(full[17])
    first = int(np.argmax(full == eos))
    gm2, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, eos_id=eos, oracle=False)
    f2 = gm2.generate_full(prompt, 40)
    s2, _ = gm2.generate(prompt, 2, 3, 40)
    np.testing.assert_array_equal(f2, full[:first + 1])
    np.testing.assert_array_equal(s2, f2)
    for tau in (0.02, 0.2):  # the adaptive loop (conditional draft passes) stops at the same token
        a2, acc, kept = gm2.generate_adaptive(prompt, 2, 3, tau, 40)
        np.testing.assert_array_equal(a2, f2)
        assert (acc <= kept).all()
    # and a handle that has stopped early generates normally afterwards
    np.testing.assert_array_equal(gm2.generate_full(prompt, 40), f2)


def test_prefill_once_decode_many():
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, 20, 1)
    B.ls_prefill(gm.h, prompt)
    B.ls_decode(gm.h, 0, 0, 30)
    full, _ = B.ls_read_output(gm.h, 30)
    for _ in range(2):
        B.ls_decode(gm.h, 2, 4, 30)
        ids, acc = B.ls_read_output(gm.h, 30)
        np.testing.assert_array_equal(ids, full)
    st = gm.stats()
    assert st.decode_ms > 0 and st.weight_bytes > 0 and st.kv_bytes > 0 and st.kernel_launches > 0
    # algorithmic bytes of the schedule: (d+1) E W_layer + d W_lm + (L-E) W_layer + W_lm per step
    s = TINY.shape
    per_step = (5 * 2 + 2) * s.layer_weight_bytes + 5 * s.lm_head_bytes
    assert st.weight_bytes == per_step * st.n_steps


def test_without_exit_cache_reuse_same_ids_more_bytes():
    """The paper's "w/o KVQ reuse" ablation: verification recomputes the early layers."""
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 128, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, 20, 1)
    B.ls_prefill(gm.h, prompt)
    B.ls_decode(gm.h, 2, 3, 40)
    ids, acc = B.ls_read_output(gm.h, 40)
    st = gm.stats()
    B.ls_decode_flags(gm.h, 2, 3, 40, B.LS_DECODE_NO_EXIT_CACHE)
    ids2, acc2 = B.ls_read_output(gm.h, 40)
    st2 = gm.stats()
    np.testing.assert_array_equal(ids2, ids)
    np.testing.assert_array_equal(acc2, acc)
    s = TINY.shape
    assert st.weight_bytes == st.n_steps * ((4 * 2 + 2) * s.layer_weight_bytes + 4 * s.lm_head_bytes)
    assert st2.weight_bytes == st2.n_steps * ((3 * 2 + 4) * s.layer_weight_bytes + 4 * s.lm_head_bytes)
    with pytest.raises(B.LsError):
        B.ls_decode_flags(gm.h, 2, 3, 40, 8)


# ------------------------------------------------------------------ odd shapes
ODD_SHAPES = [
    synth.Shape("odd-g2", 3, 104, 6, 3, 64, 200, 301),    # K = 104: ragged last k-step; 7 partial sums per row
    synth.Shape("odd-g8", 2, 128, 8, 1, 64, 344, 1000),   # 8 query heads per KV head: FMA prompt attention
    synth.Shape("odd-mha128", 2, 256, 2, 2, 128, 136, 77),  # vocabulary smaller than one prompt-GEMM tile
    synth.Shape("odd-g4", 2, 64, 4, 1, 128, 72, 513),     # q width (512) != d_model (64)
]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("shape", ODD_SHAPES, ids=lambda s: s.name)
def test_odd_shapes_logits_and_losslessness(shape, path):
    """Shapes whose sizes are not multiples of the tiles: logits against the oracle (16-row
    passes), then a 45-token prompt (tensor-core prompt pass) with every loop giving the ids
    of full greedy, which in turn follow the oracle while its margins allow."""
    gm, om = make_pair(shape, 5, 1, 0.3, 256, page_size=16, max_draft=6, linear_path=path, amplify=6.0)
    ids = synth.make_prompt(shape.vocab, 37, 3)
    gex, gfi = gm.debug_logits(ids, 1)
    oex, ofi = om.teacher_logits(ids, 1)
    assert np.abs(ofi).max() > 0.3
    assert_logits_close(gex, oex, "exit logits")
    assert_logits_close(gfi, ofi, "final logits")
    prompt = synth.make_prompt(shape.vocab, 45, 4)
    full = gm.generate_full(prompt, 40)
    for E, d in ((1, 1), (1, 3), (1, 6)):
        got, acc = gm.generate(prompt, E, d, 40)
        np.testing.assert_array_equal(got, full, err_msg=f"E={E} d={d}")
    got, acc, drafted = gm.generate_adaptive(prompt, 1, 6, 0.05, 40)
    np.testing.assert_array_equal(got, full)
    np.testing.assert_array_equal(gm.generate_early(prompt, shape.n_layers, 40), full)
    ref, margins, maxabs = om.generate_full(prompt, 40)
    k = first_low_margin(margins, maxabs)
    np.testing.assert_array_equal(full[:k], ref[:k])
    print(f"{shape.name} path {path}: ids follow the oracle for {k} of 40 tokens")
    # a prompt of more than 128 rows: the prompt GEMMs run on CTA pairs (second row tile ragged),
    # and the first token after it must be the oracle's wherever its margin allows
    long_prompt = synth.make_prompt(shape.vocab, 150, 9)
    full = gm.generate_full(long_prompt, 24)
    got, acc = gm.generate(long_prompt, 1, 3, 24)
    np.testing.assert_array_equal(got, full)
    ref, margins, maxabs = om.generate_full(long_prompt, 24)
    k = first_low_margin(margins, maxabs)
    np.testing.assert_array_equal(full[:k], ref[:k])
    print(f"{shape.name} path {path}: after a 150-token prompt the ids follow the oracle for {k} of 24 tokens")


# ------------------------------------------------------------------ the prompt pass itself
def _two_layers(shape, name):
    from dataclasses import replace
    return replace(shape, name=name, n_layers=2)


PROMPT_CASES = [(TINY.shape, 100, None), (ODD_SHAPES[0], 150, 6.0), (ODD_SHAPES[1], 150, 6.0), (ODD_SHAPES[2], 150, 6.0),
                (ODD_SHAPES[3], 150, 6.0), (_two_layers(synth.LLAMA2_7B, "7b-2-layers"), 300, None),
                (_two_layers(synth.LLAMA3_8B, "8b-2-layers"), 200, None)]


@pytest.mark.parametrize("shape,n_prompt,amp", PROMPT_CASES, ids=lambda v: getattr(v, "name", str(v)))
def test_prompt_pass_cache_gives_the_oracle_logits(shape, n_prompt, amp):
    """Next-token logits computed on top of the cache the prompt pass has left (tensor-core GEMMs
    on one CTA up to 128 rows and on CTA pairs beyond, several weight matrices per launch,
    flash-attention-style causal attention, row-wise RoPE + append) against the oracle's
    teacher-forced final logits at the last prompt position."""
    gm, om = make_pair(shape, 5, 1, 0.3, n_prompt + 8, page_size=64, max_draft=4, amplify=amp)
    prompt = synth.make_prompt(shape.vocab, n_prompt, 12)
    B.ls_prefill(gm.h, prompt)
    got = B.ls_debug_next_logits(gm.h, shape.vocab)
    _, ref = om.teacher_logits(prompt, 1)
    r = assert_logits_close(got, ref[-1], "next-token logits after the prompt pass")
    # and the 16-row passes give the same thing within the same tolerance
    _, small = gm.debug_logits(prompt, 1, want_exit=False)
    assert_logits_close(small[-1], ref[-1], "next-token logits through 16-row passes")
    print(f"{shape.name} prompt {n_prompt}: max|delta|/max|logit| {r:.2e}")


# ------------------------------------------------------------------ adaptive draft length
@pytest.mark.parametrize("path", PATHS)
def test_adaptive_equals_generate_full_for_every_threshold(path):
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, TINY.exit_layer, TINY.late_scale, 160, max_draft=15,
                      linear_path=path, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    full = gm.generate_full(prompt, TINY.max_new)
    seen = set()
    for E in (1, 2, 3):
        for d in (1, 3, 6, 15):
            for tau in (0.004, 0.02, 0.05, 0.3):
                ids, acc, drafted = gm.generate_adaptive(prompt, E, d, tau, TINY.max_new)
                np.testing.assert_array_equal(ids, full, err_msg=f"E={E} d={d} tau={tau}")
                assert ((0 <= acc) & (acc <= drafted) & (drafted <= d)).all()
                emitted = np.cumsum(acc + 1)
                assert emitted[-1] >= TINY.max_new and (len(emitted) == 1 or emitted[-2] < TINY.max_new)
                st = gm.stats()
                assert st.n_steps == len(acc) and st.n_accepted == acc.sum() and st.host_syncs <= 10
                seen.update(drafted.tolist())
    assert {0, 1, 2, 3, 6, 15} <= seen  # stops at once, in the middle, and never


@pytest.mark.parametrize("path", PATHS)
def test_adaptive_limits_are_the_fixed_loop_and_one_token_per_step(path):
    E, d = TINY.exit_layer, 5
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 128, linear_path=path, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    ids0, acc0 = gm.generate(prompt, E, d, 40)
    w0 = gm.stats().weight_bytes
    ids, acc, drafted = gm.generate_adaptive(prompt, E, d, 1e-30, 40)  # no margin is below it
    np.testing.assert_array_equal(ids, ids0)
    np.testing.assert_array_equal(acc, acc0)
    assert (drafted == d).all() and gm.stats().weight_bytes == w0
    ids, acc, drafted = gm.generate_adaptive(prompt, E, d, float("inf"), 40)  # every margin is below it
    np.testing.assert_array_equal(ids, ids0)
    assert len(acc) == 40 and (acc == 0).all() and (drafted == 0).all()
    # one early pass + its head + the verify of one row per step: the bytes of plain greedy
    s = TINY.shape
    assert gm.stats().weight_bytes == 40 * (s.n_layers * s.layer_weight_bytes + 2 * s.lm_head_bytes)
    np.testing.assert_array_equal(B.ls_read_drafted(gm.h, 40), drafted)
    for bad in (0.0, -1.0, float("nan")):
        with pytest.raises(B.LsError) as e:
            gm.generate_adaptive(prompt, E, d, bad, 40)
        assert e.value.status == B.LS_ERR_INVALID_ARG
    gm.generate(prompt, E, d, 40)
    assert (B.ls_read_drafted(gm.h, 40) == d).all()  # the fixed loop keeps d drafts every step


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("tau", [0.02, 0.05])
def test_adaptive_steps_follow_the_oracle_margins(path, tau):
    """Every step's kept-draft count k and accepted count n, checked against the oracle's exit
    logits.  The ids are the full model's, so the state a step starts from is known from the
    number of tokens emitted before it; from there the oracle replays the draft chain.  A step
    is compared when all its decisions are clear: every margin the chain meets is further from
    the threshold (and from zero, for the draft token itself) than the two sides can differ.
    A margin is the difference of two logits, so that distance is 2 max|logit error|, the
    error measured on the teacher-forced exit logits of the same sequence (itself held to the
    logit tolerance), doubled once more for drafts that leave that sequence."""
    E, d, new = TINY.exit_layer, 4, TINY.max_new
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 128, linear_path=path)
    prompt = synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, TINY.prompt_seed)
    full = gm.generate_full(prompt, new + d + 1)
    ids, acc, drafted = gm.generate_adaptive(prompt, E, d, tau, new)
    np.testing.assert_array_equal(ids, full[:new])
    seq_all = np.concatenate([prompt, full])
    ex, _ = om.teacher_logits(seq_all, E)
    gex, _ = gm.debug_logits(seq_all, E, want_final=False)
    assert_logits_close(gex, ex, "exit logits")
    tol = 2 * 2 * np.abs(gex - ex).max()
    emitted = checked = 0
    for k_gpu, n_gpu in zip(drafted, acc):
        seq, drafts, clear, k_ref = list(prompt) + list(full[:emitted]), [], True, d
        for j in range(d):
            z = om.teacher_logits(np.array(seq + drafts, dtype=np.int32), E)[0][-1]
            top = np.sort(z)[-2:]
            margin = top[1] - top[0]
            if abs(margin - tau) <= tol:
                clear = False
                break
            if margin < tau:
                k_ref = j
                break
            drafts.append(int(z.argmax()))
        if clear:
            n_ref = 0
            while n_ref < k_ref and drafts[n_ref] == full[emitted + n_ref]:
                n_ref += 1
            assert (k_gpu, n_gpu) == (k_ref, n_ref), f"step starting after {emitted} tokens"
            checked += 1
        emitted += n_gpu + 1
    print(f"path {path} tau {tau}: {checked} of {len(acc)} steps clear and equal; kept/step {drafted.mean():.2f}, "
          f"margin tolerance {tol:.2e}")
    assert checked >= len(acc) // 2


def test_boundary_error_codes():
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 64, max_draft=4, oracle=False)
    p = synth.make_prompt(TINY.shape.vocab, 8, 0)

    def status(fn, *a):
        with pytest.raises(B.LsError) as e:
            fn(*a)
        return e.value.status

    assert status(gm.generate, p, 4, 2, 8) == B.LS_ERR_INVALID_ARG       # E must leave a layer to verify with
    assert status(gm.generate, p, 0, 2, 8) == B.LS_ERR_INVALID_ARG
    assert status(gm.generate, p, 2, 5, 8) == B.LS_ERR_CAPACITY          # beyond max_draft
    assert status(gm.generate, p, 2, 2, 60) == B.LS_ERR_CAPACITY         # KV capacity
    assert status(gm.generate_full, p, 60) == B.LS_ERR_CAPACITY
    bad = p.copy()
    bad[3] = TINY.shape.vocab
    assert status(gm.generate_full, bad, 4) == B.LS_ERR_INVALID_ARG
    assert status(gm.generate_full, p[:0], 4) == B.LS_ERR_INVALID_ARG
    # the handle is still usable after every refusal
    assert len(gm.generate_full(p, 4)) == 4
    cfg = B.make_config(TINY.shape, 64)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.LsError) as e:
        B.ls_model_create(cfg, gm.weights, ws)
    assert e.value.status == B.LS_ERR_CAPACITY


@pytest.mark.parametrize("path", PATHS)
def test_exactly_at_kv_capacity(path):
    """n_prompt + max_new + d + 1 == max_seq: the last step's rows reach the last cache
    position (the chunked attention's last, partly filled chunk; page 3 of 4 pages of 16)."""
    d = 3
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 64, page_size=16, max_draft=d,
                      linear_path=path, oracle=False)
    prompt = synth.make_prompt(TINY.shape.vocab, 20, 6)
    full = gm.generate_full(prompt, 40)
    ids, acc = gm.generate(prompt, 2, d, 40)          # 20 + 40 + 3 + 1 = 64
    np.testing.assert_array_equal(ids, full)
    ids, acc, kept = gm.generate_adaptive(prompt, 2, d, 0.05, 40)
    np.testing.assert_array_equal(ids, full)
    with pytest.raises(B.LsError) as e:
        gm.generate(prompt, 2, d, 41)
    assert e.value.status == B.LS_ERR_CAPACITY
    assert len(gm.generate_full(prompt, 43)) == 43    # 20 + 43 + 1 = 64 for plain greedy


# ------------------------------------------------------------------ Llama-2-7B shape
@pytest.fixture(scope="module")
def llama7b():
    wl = synth.WORKLOADS["llama2-7b"]
    max_seq = wl.n_prompt + wl.max_new + wl.num_draft + 1
    w = synth.make_weights(wl.shape, wl.weight_seed, wl.exit_layer, wl.late_scale, device="cuda")
    gm = B.Model(wl.shape, w, max_seq, 64, 8)
    yield wl, gm, w
    gm.close()


def test_llama7b_generate_equals_generate_full_at_full_size(llama7b):
    """The benchmark's configuration: prompt 1024, 256 new tokens, E=8, d=6."""
    wl, gm, _ = llama7b
    prompt = synth.make_prompt(wl.shape.vocab, wl.n_prompt, wl.prompt_seed)
    full = gm.generate_full(prompt, wl.max_new)
    t_full = gm.stats().decode_ms
    ids, acc = gm.generate(prompt, wl.exit_layer, wl.num_draft, wl.max_new)
    st = gm.stats()
    np.testing.assert_array_equal(ids, full)
    assert len(ids) == wl.max_new and np.cumsum(acc + 1)[-1] >= wl.max_new
    assert ((0 <= acc) & (acc <= wl.num_draft)).all()
    print(f"7B: full {wl.max_new / t_full * 1e3:.1f} tok/s, self-spec {wl.max_new / st.decode_ms * 1e3:.1f} tok/s, "
          f"accepted/step {acc.mean():.2f}, syncs {st.host_syncs}")


def test_llama7b_logits_against_oracle_on_a_short_prompt(llama7b):
    """What the oracle can afford at this shape: 17 teacher-forced positions (a 16-row pass and
    a single-row pass through all 32 layers)."""
    from oracle import ls_oracle as O
    wl, gm, w = llama7b
    s = wl.shape
    cfg = O.Config(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab,
                   s.rms_eps, s.rope_theta, 24)
    om = O.Model(cfg, synth.as_uint16(w))
    ids = synth.make_prompt(s.vocab, 17, 17)
    oex, ofi = om.teacher_logits(ids, wl.exit_layer)
    gex, gfi = gm.debug_logits(ids, wl.exit_layer)
    r1 = assert_logits_close(gex, oex, "exit logits")
    r2 = assert_logits_close(gfi, ofi, "final logits")
    for g, o in ((gex, oex), (gfi, ofi)):
        part = np.partition(o, -2, axis=1)
        safe = (part[:, -1] - part[:, -2]) > LOGIT_TOL * np.abs(o).max()
        assert (g.argmax(1)[safe] == o.argmax(1)[safe]).all()
    print(f"7B: max|delta|/max|logit| exit {r1:.2e} final {r2:.2e}; max|logit| {np.abs(ofi).max():.3f}")
