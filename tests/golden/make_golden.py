"""Writes tests/golden/tiny_workload.json.  Calls ONLY the CPU oracle (and the seeded input
generators): no value in the fixture ever comes from the CUDA path.

    python tests/golden/make_golden.py

The fixture holds, for the `tiny` workload with weights drawn on the CPU: the full-model greedy
ids with their top-1/top-2 margins, the self-speculative accepted-per-step counts for
(E, d) = (2, 3), early-exit ids, and teacher-forced exit / final logits of the first 12 prompt
ids at eight vocabulary indices.  There is no worked numeric example in the paper to store
(it prints only throughput and quality tables), so these are the oracle's own values, kept to
notice any later change of its arithmetic and to give the GPU tests a reference that is not
recomputed on the spot.
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ls_oracle as O  # noqa: E402
from paper_2404_16710_b200 import synth  # noqa: E402


def main():
    wl = synth.WORKLOADS["tiny"]
    s = wl.shape
    w = synth.as_uint16(synth.make_weights(s, wl.weight_seed, wl.exit_layer, wl.late_scale, device="cpu"))
    m = O.Model(O.Config(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab, s.rms_eps,
                         s.rope_theta, 128), w)
    prompt = synth.make_prompt(s.vocab, wl.n_prompt, wl.prompt_seed)
    full, margins, maxabs = m.generate_full(prompt, wl.max_new)
    ids, acc, trace = m.generate_spec(prompt, wl.exit_layer, wl.num_draft, wl.max_new)
    early = m.generate_early(prompt, wl.exit_layer, 16)
    assert (ids == full).all()
    # teacher-forced logits of the first 12 prompt ids at 8 fixed vocabulary indices
    cols = [0, 1, 17, 255, 256, 511, 700, s.vocab - 1]
    ex, fi = m.teacher_logits(prompt[:12], wl.exit_layer)
    out = {"workload": "tiny", "weights": "synth.make_weights(device='cpu')", "prompt": prompt.tolist(),
           "exit_layer": wl.exit_layer, "num_draft": wl.num_draft, "full_greedy_ids": full.tolist(),
           "margins": [round(float(x), 9) for x in margins], "max_abs_logit": [round(float(x), 9) for x in maxabs],
           "accepted_per_step": acc.tolist(), "cache_len_after_step": trace.tolist(), "early_exit_ids": early.tolist(),
           "logit_columns": cols, "exit_logits": [[round(float(v), 9) for v in row] for row in ex[:, cols]],
           "final_logits": [[round(float(v), 9) for v in row] for row in fi[:, cols]],
           "max_abs_final_logit": round(float(abs(fi).max()), 9), "max_abs_exit_logit": round(float(abs(ex).max()), 9)}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_workload.json"), "w") as f:
        json.dump(out, f, indent=1)
    print("wrote tiny_workload.json:", len(full), "ids,", len(acc), "steps")


if __name__ == "__main__":
    main()
