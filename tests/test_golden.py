"""Stored expected values (tests/golden/tiny_workload.json, written by tests/golden/make_golden.py from the
oracle alone): the oracle must still reproduce them exactly; the CUDA path must match them on the prefix
whose margins exceed the logits tolerance."""
import json
import os

import numpy as np
import pytest

from oracle import ls_oracle as O
from paper_2404_16710_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_workload.json")))
WL = synth.WORKLOADS["tiny"]


def cpu_weights():
    return synth.make_weights(WL.shape, WL.weight_seed, WL.exit_layer, WL.late_scale, device="cpu")


def test_oracle_reproduces_the_stored_values():
    s = WL.shape
    m = O.Model(O.Config(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab, s.rms_eps,
                         s.rope_theta, 128), synth.as_uint16(cpu_weights()))
    prompt = np.asarray(GOLD["prompt"], dtype=np.int32)
    np.testing.assert_array_equal(prompt, synth.make_prompt(s.vocab, WL.n_prompt, WL.prompt_seed))
    full, margins, maxabs = m.generate_full(prompt, WL.max_new)
    np.testing.assert_array_equal(full, GOLD["full_greedy_ids"])
    np.testing.assert_allclose(margins, GOLD["margins"], rtol=0, atol=1e-8)
    ids, acc, trace = m.generate_spec(prompt, GOLD["exit_layer"], GOLD["num_draft"], WL.max_new)
    np.testing.assert_array_equal(ids, GOLD["full_greedy_ids"])
    np.testing.assert_array_equal(acc, GOLD["accepted_per_step"])
    np.testing.assert_array_equal(trace, GOLD["cache_len_after_step"])
    np.testing.assert_array_equal(m.generate_early(prompt, GOLD["exit_layer"], 16), GOLD["early_exit_ids"])
    ex, fi = m.teacher_logits(prompt[:12], GOLD["exit_layer"])
    np.testing.assert_allclose(ex[:, GOLD["logit_columns"]], GOLD["exit_logits"], rtol=0, atol=1e-8)
    np.testing.assert_allclose(fi[:, GOLD["logit_columns"]], GOLD["final_logits"], rtol=0, atol=1e-8)


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_values_on_the_safe_prefix():
    from paper_2404_16710_b200 import binding as B
    w = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in cpu_weights().items()}
    gm = B.Model(WL.shape, w, 128, 64, 8)
    prompt = np.asarray(GOLD["prompt"], dtype=np.int32)
    margins, maxabs = np.asarray(GOLD["margins"]), np.asarray(GOLD["max_abs_logit"])
    low = np.nonzero(margins <= 3e-2 * maxabs)[0]
    k = int(low[0]) if low.size else len(margins)
    assert k >= 1
    gex, gfi = gm.debug_logits(prompt[:12], GOLD["exit_layer"])
    cols = GOLD["logit_columns"]
    assert np.abs(gex[:, cols] - np.asarray(GOLD["exit_logits"])).max() <= 3e-2 * GOLD["max_abs_exit_logit"]
    assert np.abs(gfi[:, cols] - np.asarray(GOLD["final_logits"])).max() <= 3e-2 * GOLD["max_abs_final_logit"]
    ids, acc = gm.generate(prompt, GOLD["exit_layer"], GOLD["num_draft"], WL.max_new)
    full = gm.generate_full(prompt, WL.max_new)
    np.testing.assert_array_equal(ids, full)
    np.testing.assert_array_equal(ids[:k], GOLD["full_greedy_ids"][:k])
