"""Several sequences per pass (ls_generate_batch): every sequence against its own
single-sequence runs and against the oracle.

The oracle needs nothing new: B sequences are B independent runs of the paper's loop
(Appendix A.4).  What the library adds is that the B sequences share every pass, and with it
every weight read; the tests check that sharing changes no bit of any sequence.
"""
import numpy as np
import pytest

from paper_2404_16710_b200 import binding as B
from paper_2404_16710_b200 import synth
from tests.helpers import LOGIT_TOL, make_pair
from tests.test_gpu_parity_configs import clear_steps_equal, rel_margins

pytestmark = pytest.mark.gpu
PATHS = [B.LS_LINEAR_FMA, B.LS_LINEAR_MMA]
TINY = synth.WORKLOADS["tiny"]
ODD_G2 = synth.Shape("odd-g2", 3, 104, 6, 3, 64, 200, 301)


def prompts_of(shape, lens, seed):
    return [synth.make_prompt(shape.vocab, n, seed + i) for i, n in enumerate(lens)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("shape,E,d,lens,new", [
    (TINY.shape, 2, 3, (32, 9, 70, 17), 40),      # 4 sequences x 4 rows = the 16 rows of a pass
    (TINY.shape, 1, 7, (33, 64), 35),             # 2 x 8 rows
    (TINY.shape, 3, 1, (5, 6, 7, 8, 9, 10, 11, 12), 20),
    (ODD_G2, 1, 2, (40, 3, 129), 25),             # grouped heads, dims off the tile sizes
    (TINY.shape, 2, 2, (150,), 30),               # a batch of one
], ids=lambda v: getattr(v, "name", str(v)))
def test_every_sequence_equals_its_own_single_sequence_runs(path, shape, E, d, lens, new):
    """ids of sequence b == ls_generate_full(prompt b) == ls_generate(prompt b), bit for bit,
    and accepted-per-step == ls_generate's: a row's arithmetic does not depend on which other
    rows share its pass."""
    cap = max(lens) + new + d + 2
    max_seq = len(lens) * (-(-cap // 16) * 16)
    gm, _ = make_pair(shape, 77, E, 0.1, max_seq, page_size=16, max_draft=d, linear_path=path, amplify=6.0)
    prompts = prompts_of(shape, lens, 500)
    got = gm.generate_batch(prompts, E, d, new)
    assert len(got) == len(lens)
    for p, (ids, acc) in zip(prompts, got):
        full = gm.generate_full(p, new)
        ids1, acc1 = gm.generate(p, E, d, new)
        np.testing.assert_array_equal(ids, full)
        np.testing.assert_array_equal(ids1, full)
        np.testing.assert_array_equal(acc, acc1)
        assert len(ids) == new and (acc.sum() + len(acc)) >= new
    # the call after a batch starts from a clean state, and a second batch repeats the first
    again = gm.generate_batch(prompts, E, d, new)
    for (a, b), (c, e) in zip(got, again):
        np.testing.assert_array_equal(a, c)
        np.testing.assert_array_equal(b, e)


@pytest.mark.parametrize("path", PATHS)
def test_batched_plain_greedy_equals_single_sequence_greedy(path):
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 4 * 96, page_size=32, max_draft=3,
                      linear_path=path)
    prompts = prompts_of(TINY.shape, (20, 31, 8, 50), 900)
    got = gm.generate_batch(prompts, 0, 0, 24)
    for p, (ids, acc) in zip(prompts, got):
        np.testing.assert_array_equal(ids, gm.generate_full(p, 24))
        assert (acc == 0).all() and len(acc) == 24


@pytest.mark.parametrize("path", PATHS)
def test_batch_sequences_against_the_oracle(path):
    """Per sequence, as for a single one: ids equal the oracle's on the safe-margin prefix, and
    every step whose rows are clear of the logit tolerance accepts what the oracle's logits
    say (Appendix A.4's match)."""
    E, d, new = TINY.exit_layer, TINY.num_draft, 48
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 4 * 128, page_size=64, max_draft=d,
                       linear_path=path)
    prompts = [synth.make_prompt(TINY.shape.vocab, TINY.n_prompt, s) for s in (141, 87, TINY.prompt_seed, 7)]
    got = gm.generate_batch(prompts, E, d, new)
    checked_total = steps_total = 0
    for p, (ids, acc) in zip(prompts, got):
        ref, margins, maxabs = om.generate_full(p, new)
        low = np.nonzero(margins <= LOGIT_TOL * maxabs)[0]
        k = int(low[0]) if low.size else new
        np.testing.assert_array_equal(ids[:k], ref[:k])
        checked, steps, _ = clear_steps_equal(gm, om, p, E, d, ids, acc)
        checked_total += checked
        steps_total += steps
    assert checked_total >= steps_total // 4


def test_batch_on_the_7b_layer_shapes():
    """Two layers of the Llama-2-7B shape, 4 sequences x 4 rows and 8 x 2 rows: the passes of 9 to 16
    rows run the per-SM cut of the o-proj and down-proj matrices, the single-sequence runs the
    tile-per-CTA cut; every sequence must still equal its own greedy run bit for bit."""
    from dataclasses import replace
    shape = replace(synth.LLAMA2_7B, name="7b-2-layers", n_layers=2)
    gm, _ = make_pair(shape, 1234, 1, 0.05, 8 * 128, page_size=64, max_draft=3, oracle=False)
    prompts = prompts_of(shape, (40, 90, 17, 64, 33, 100, 5, 71), 77)
    for nb, d in ((4, 3), (8, 1)):
        got = gm.generate_batch(prompts[:nb], 1, d, 20)
        for p, (ids, acc) in zip(prompts, got):
            np.testing.assert_array_equal(ids, gm.generate_full(p, 20))
            ids1, acc1 = gm.generate(p, 1, d, 20)
            np.testing.assert_array_equal(ids1, ids)
            np.testing.assert_array_equal(acc1, acc)


def test_batch_zero_late_scale_accepts_every_draft():
    """Late layers that add nothing: draft == verified at every row of every sequence, so each
    step accepts d drafts whatever the sequence (the oracle's closed-form case)."""
    E, d = 2, 3
    gm, om = make_pair(TINY.shape, TINY.weight_seed, E, 0.0, 4 * 64, page_size=16, max_draft=d)
    prompts = prompts_of(TINY.shape, (10, 14, 3, 21), 40)
    for p, (ids, acc) in zip(prompts, gm.generate_batch(prompts, E, d, 22)):
        oids, oacc, _ = om.generate_spec(p, E, d, 22)
        np.testing.assert_array_equal(acc, oacc)
        assert (acc == d).all()


def test_batch_sequences_stop_on_their_own():
    """EOS ends one sequence while the others continue to max_new."""
    E, d, new = 2, 3, 30
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 3 * 96, page_size=32, max_draft=d)
    prompts = prompts_of(TINY.shape, (12, 25, 18), 321)
    free = gm.generate_batch(prompts, E, d, new)
    eos = int(free[1][0][7])  # the 8th token of sequence 1 becomes the end-of-sequence id
    gm2, _ = make_pair(TINY.shape, TINY.weight_seed, E, TINY.late_scale, 3 * 96, page_size=32, max_draft=d, eos_id=eos)
    for b, (ids, acc) in enumerate(gm2.generate_batch(prompts, E, d, new)):
        ref = free[b][0]
        hit = np.nonzero(ref == eos)[0]
        n = int(hit[0]) + 1 if hit.size else new
        np.testing.assert_array_equal(ids, ref[:n])
        np.testing.assert_array_equal(ids, gm2.generate_full(prompts[b], new))


def test_batch_argument_errors():
    gm, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 256, page_size=64, max_draft=3)
    p = prompts_of(TINY.shape, (8, 8, 8, 8, 8), 1)
    with pytest.raises(B.LsError) as e:
        gm.generate_batch(p, 2, 3, 8)          # 5 x 4 rows > 16
    assert e.value.status == B.LS_ERR_CAPACITY
    with pytest.raises(B.LsError) as e:
        gm.generate_batch(p[:4], 2, 3, 60)     # 64 positions per sequence: 8 + 60 + 4 > 64
    assert e.value.status == B.LS_ERR_CAPACITY
    with pytest.raises(B.LsError) as e:
        gm.generate_batch(p[:2], 4, 3, 8)      # exit layer must leave a late layer
    assert e.value.status == B.LS_ERR_INVALID_ARG
    with pytest.raises(B.LsError) as e:
        gm.generate_batch(p[:2], 0, 2, 8)
    assert e.value.status == B.LS_ERR_INVALID_ARG
    fresh, _ = make_pair(TINY.shape, TINY.weight_seed, 2, TINY.late_scale, 256, page_size=64, max_draft=3, oracle=False)
    with pytest.raises(B.LsError) as e:
        B.ls_decode_batch(fresh.h, 2, 3, 8)    # nothing prefilled
    assert e.value.status == B.LS_ERR_INVALID_ARG
    bad = [np.array([1, 2, TINY.shape.vocab], dtype=np.int32)]
    with pytest.raises(B.LsError) as e:
        gm.generate_batch(bad, 2, 3, 8)
    assert e.value.status == B.LS_ERR_INVALID_ARG
    ids, acc = gm.generate_batch(p[:2], 2, 3, 8)[1]  # the handle is still good
    np.testing.assert_array_equal(ids, gm.generate_full(p[1], 8))
