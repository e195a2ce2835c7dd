"""Pins for the oracle's model-level routines.  CPU only.

* the cached token-by-token C forward equals a numpy recomputation without any
  cache (full [T, T] attention matrices) -- logits at the exit layer and at the top;
* greedy / early-exit generation equal the no-cache greedy recomputation;
* grouped KV heads: replicating the KV heads into an MHA model changes nothing;
* exit logits at E = L are the final logits;
* losslessness (Sec. 4.3 of the paper: verification keeps exactly the full model's
  tokens): self-speculative ids == full greedy ids for EVERY (E, d);
* zero late-layer scale: x_L = x_E, so every draft is accepted (n == d each step);
* bookkeeping invariants of the loop in Appendix A.4;
* the adaptive-draft-length extension: same ids as full greedy for every threshold, the two
  limits (threshold -> 0: the fixed-length loop; +inf: one token per step), and every step's
  kept-draft and accepted counts re-derived from no-cache exit logits.
"""
from dataclasses import replace

import numpy as np
import pytest

from oracle import ls_bruteforce as B
from oracle import ls_oracle as O
from paper_2404_16710_b200 import synth


def oracle_model(shape, seed=7, scale_from=0, late_scale=1.0, max_seq=96, eos_id=-1, weights=None):
    w = weights or synth.as_uint16(synth.make_weights(shape, seed, scale_from, late_scale))
    cfg = O.Config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                   shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta, max_seq, eos_id)
    return O.Model(cfg, w), cfg, w


# N(0, 0.02) weights on a 64-wide model give nearly flat logits; a larger draw makes
# the comparisons below sensitive to every term.
def loud_weights(shape, seed=11):
    w = synth.make_weights(shape, seed, 0, 1.0)
    for k, v in w.items():
        if k in ("attn_norm", "ffn_norm", "final_norm"):
            continue
        if isinstance(v, list):
            w[k] = [(t.float() * 6).bfloat16() for t in v]
        else:
            w[k] = (v.float() * 6).bfloat16()
    return synth.as_uint16(w)


@pytest.mark.parametrize("shape", [synth.MICRO_GQA, synth.MICRO_MHA], ids=lambda s: s.name)
@pytest.mark.parametrize("E", [1, 2])
def test_cached_forward_equals_no_cache_recomputation(shape, E):
    m, cfg, w = oracle_model(shape, weights=loud_weights(shape))
    ids = synth.make_prompt(shape.vocab, 13, 5)
    ex, fi = m.teacher_logits(ids, E)
    np.testing.assert_allclose(ex, B.logits_at(cfg, w, ids, E), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(fi, B.logits_at(cfg, w, ids, shape.n_layers), rtol=1e-9, atol=1e-11)
    assert np.abs(fi).max() > 0.1  # the comparison is not vacuous


@pytest.mark.parametrize("first", [0, 5, 12, 13])
def test_teacher_logits_tail_equals_no_cache_recomputation(first):
    """Logits asked for the last positions only: the rows of the no-cache recomputation at those
    positions (and the earlier positions still fill the cache: the rows would differ otherwise)."""
    shape = synth.MICRO_GQA
    m, cfg, w = oracle_model(shape, weights=loud_weights(shape))
    ids = synth.make_prompt(shape.vocab, 13, 5)
    ex, fi = m.teacher_logits_tail(ids, 2, first)
    assert ex.shape == fi.shape == (13 - first, shape.vocab)
    np.testing.assert_allclose(ex, B.logits_at(cfg, w, ids, 2)[first:], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(fi, B.logits_at(cfg, w, ids, shape.n_layers)[first:], rtol=1e-9, atol=1e-11)
    with pytest.raises(ValueError):
        m.teacher_logits_tail(ids, 2, 14)


def test_greedy_and_early_exit_equal_no_cache_greedy():
    shape = synth.MICRO_GQA
    m, cfg, w = oracle_model(shape, weights=loud_weights(shape))
    prompt = synth.make_prompt(shape.vocab, 6, 9)
    ids, margins, maxabs = m.generate_full(prompt, 10)
    np.testing.assert_array_equal(ids, B.greedy(cfg, w, prompt, 10))
    assert margins.min() > 1e-6 and maxabs.min() > 0
    np.testing.assert_array_equal(m.generate_early(prompt, 2, 10), B.greedy(cfg, w, prompt, 10, layer=2))


def test_grouped_kv_heads_equal_replicated_mha():
    g = synth.MICRO_GQA
    wg = loud_weights(g)
    rep = g.n_heads // g.n_kv_heads
    wm = dict(wg)
    for name in ("wk", "wv"):
        wm[name] = [np.ascontiguousarray(
            np.repeat(a.reshape(g.n_kv_heads, g.head_dim, g.d_model), rep, axis=0)
            .reshape(g.n_heads * g.head_dim, g.d_model)) for a in wg[name]]
    mha = replace(g, n_kv_heads=g.n_heads)
    ids = synth.make_prompt(g.vocab, 9, 2)
    a = oracle_model(g, weights=wg)[0].teacher_logits(ids, 1)
    b = oracle_model(mha, weights=wm)[0].teacher_logits(ids, 1)
    np.testing.assert_allclose(a[0], b[0], rtol=1e-12)
    np.testing.assert_allclose(a[1], b[1], rtol=1e-12)


def test_exit_logits_at_last_layer_are_the_final_logits():
    shape = synth.MICRO_MHA
    m, _, _ = oracle_model(shape)
    ex, fi = m.teacher_logits(synth.make_prompt(shape.vocab, 7, 3), shape.n_layers)
    np.testing.assert_array_equal(ex, fi)


@pytest.mark.parametrize("E,d", [(E, d) for E in (1, 2, 3) for d in (1, 2, 3, 5)])
def test_losslessness_tiny_every_exit_and_draft(E, d):
    wl = synth.WORKLOADS["tiny"]
    m, _, _ = oracle_model(wl.shape, wl.weight_seed, E, wl.late_scale, max_seq=96)
    prompt = synth.make_prompt(wl.shape.vocab, 12, wl.prompt_seed)
    full, _, _ = m.generate_full(prompt, 24)
    ids, acc, trace = m.generate_spec(prompt, E, d, 24)
    np.testing.assert_array_equal(ids, full)
    # cache length after each step = P - 1 + tokens emitted so far (untruncated)
    np.testing.assert_array_equal(trace, len(prompt) - 1 + np.cumsum(acc + 1))
    assert ((0 <= acc) & (acc <= d)).all()
    emitted = np.cumsum(acc + 1)
    assert emitted[-1] >= 24 and (len(emitted) == 1 or emitted[-2] < 24)  # only the last step truncates


def test_losslessness_micro_gqa_loud_weights():
    shape = synth.MICRO_GQA
    m, _, _ = oracle_model(shape, weights=loud_weights(shape))
    prompt = synth.make_prompt(shape.vocab, 5, 1)
    full, _, _ = m.generate_full(prompt, 20)
    for E in (1, 2):
        for d in (1, 4):
            ids, acc, _ = m.generate_spec(prompt, E, d, 20)
            np.testing.assert_array_equal(ids, full)
    assert len(set(full.tolist())) > 3  # not a degenerate repetition of one token


def test_zero_late_scale_accepts_every_draft():
    wl = synth.WORKLOADS["tiny"]
    E, d = 2, 3
    m, _, _ = oracle_model(wl.shape, wl.weight_seed, E, 0.0, max_seq=96)
    prompt = synth.make_prompt(wl.shape.vocab, 10, wl.prompt_seed)
    ids, acc, trace = m.generate_spec(prompt, E, d, 22)
    assert (acc == d).all()
    assert len(acc) == -(-22 // (d + 1))
    np.testing.assert_array_equal(ids, m.generate_full(prompt, 22)[0])
    # and the full model's tokens are then the early-exit tokens
    np.testing.assert_array_equal(ids, m.generate_early(prompt, E, 22))


def test_acceptance_falls_as_late_layers_grow():
    wl = synth.WORKLOADS["tiny"]
    prompt = synth.make_prompt(wl.shape.vocab, 10, wl.prompt_seed)
    mean_acc = []
    for s in (0.0, 0.1, 3.0):
        m, _, _ = oracle_model(wl.shape, wl.weight_seed, 2, s, max_seq=96)
        _, acc, _ = m.generate_spec(prompt, 2, 3, 30)
        mean_acc.append(acc.mean())
    assert mean_acc[0] == 3.0 and mean_acc[0] >= mean_acc[1] >= mean_acc[2] and mean_acc[2] < 3.0


def test_eos_stops_both_loops_at_the_same_token():
    wl = synth.WORKLOADS["tiny"]
    m, _, _ = oracle_model(wl.shape, wl.weight_seed, 2, wl.late_scale, max_seq=96)
    prompt = synth.make_prompt(wl.shape.vocab, 12, wl.prompt_seed)
    full, _, _ = m.generate_full(prompt, 24)
    eos = int(full[9])
    first = int(np.argmax(full == eos))
    m2, _, _ = oracle_model(wl.shape, wl.weight_seed, 2, wl.late_scale, max_seq=96, eos_id=eos)
    f2, _, _ = m2.generate_full(prompt, 24)
    s2, _, _ = m2.generate_spec(prompt, 2, 3, 24)
    np.testing.assert_array_equal(f2, full[:first + 1])
    np.testing.assert_array_equal(s2, f2)


# ---------------------------------------------------------------- adaptive draft length
def tiny_model(E, late_scale=None, max_seq=96):
    wl = synth.WORKLOADS["tiny"]
    m, cfg, w = oracle_model(wl.shape, wl.weight_seed, E, wl.late_scale if late_scale is None else late_scale,
                             max_seq=max_seq)
    return m, cfg, w, synth.make_prompt(wl.shape.vocab, 12, wl.prompt_seed)


@pytest.mark.parametrize("E,d", [(1, 3), (2, 4), (3, 2)])
@pytest.mark.parametrize("tau", [0.004, 0.02, 0.05, 0.3])
def test_adaptive_is_lossless_for_every_threshold(E, d, tau):
    m, _, _, prompt = tiny_model(E)
    full, _, _ = m.generate_full(prompt, 24)
    ids, acc, drafted, _ = m.generate_adaptive(prompt, E, d, tau, 24)
    np.testing.assert_array_equal(ids, full)
    assert ((0 <= acc) & (acc <= drafted) & (drafted <= d)).all()
    emitted = np.cumsum(acc + 1)
    assert emitted[-1] >= 24 and (len(emitted) == 1 or emitted[-2] < 24)


def test_adaptive_limits_are_the_fixed_loop_and_one_token_per_step():
    E, d = 2, 4
    m, _, _, prompt = tiny_model(E)
    ids0, acc0, _ = m.generate_spec(prompt, E, d, 24)
    ids, acc, drafted, gap = m.generate_adaptive(prompt, E, d, 1e-300, 24)  # no margin is below it
    np.testing.assert_array_equal(ids, ids0)
    np.testing.assert_array_equal(acc, acc0)
    assert (drafted == d).all() and gap.min() > 0
    ids, acc, drafted, _ = m.generate_adaptive(prompt, E, d, np.inf, 24)  # every margin is below it
    np.testing.assert_array_equal(ids, ids0)
    assert len(acc) == 24 and (acc == 0).all() and (drafted == 0).all()
    with pytest.raises(ValueError):
        m.generate_adaptive(prompt, E, d, 0.0, 24)


@pytest.mark.parametrize("tau", [0.02, 0.05])
def test_adaptive_steps_rederived_from_no_cache_exit_logits(tau):
    """Each step's kept-draft count k and accepted count n, recomputed without any cache:
    the exit logits of the growing sequence (full [T, T] attention) give the margins and the
    drafts; n is the agreement of those drafts with the full model's greedy continuation."""
    E, d, new = 2, 4, 18
    m, cfg, w, prompt = tiny_model(E)
    ids, acc, drafted, _ = m.generate_adaptive(prompt, E, d, tau, new)
    full = B.greedy(cfg, w, prompt, new + d + 1)
    np.testing.assert_array_equal(ids, full[:new])
    emitted = 0
    for k_ref, n_ref in zip(drafted, acc):
        seq = list(prompt) + list(full[:emitted])
        drafts = []
        k = d
        for j in range(d):
            z = B.logits_at(cfg, w, np.array(seq + drafts, dtype=np.int32), E)[-1]
            top = np.sort(z)[-2:]
            if top[1] - top[0] < tau:
                k = j
                break
            drafts.append(int(z.argmax()))
        n = 0
        while n < k and drafts[n] == full[emitted + n]:
            n += 1
        assert (k, n) == (k_ref, n_ref)
        emitted += n + 1
    assert emitted >= new
    assert 0 < drafted.mean() < d  # the threshold bites, and not always at once


def test_argument_errors():
    shape = synth.MICRO_MHA
    m, _, _ = oracle_model(shape, max_seq=32)
    p = synth.make_prompt(shape.vocab, 4, 0)
    with pytest.raises(ValueError):
        m.generate_spec(p, shape.n_layers, 2, 4)   # E must leave a layer to verify with
    with pytest.raises(ValueError):
        m.generate_spec(p, 1, 2, 32)               # would overflow the cache
    with pytest.raises(ValueError):
        m.generate_full(p, 40)
