"""Timeline of one decode pass inside the loop: when each kernel's CTAs start, when its
dependency wait is released and when it ends, relative to the kernel before it.

    python -m paper_2404_16710_b200.build --trace          # libls_b200_trace.so (-DLS_TRACE)
    python -m paper_2404_16710_b200.timeline --workload llama2-7b [--spec] [--layers 4,20]

The kernels of the loop are chained by programmatic dependent launch, so their lifetimes
overlap and per-kernel durations from a profiler (which serialises launches) do not add up
to the loop's time.  The trace build stamps the global timer inside the linear and attention
kernels (see ls_common.cuh); this driver runs one full-greedy token (or one self-speculative
step with --spec) with recording on and prints, per launch: first / last CTA start, first /
last release of the dependency wait, first / last CTA end, the time from the previous kernel's
end to this kernel's end, and the gap between the previous kernel's end and the release.
Recording costs a few percent of the pass; the product library carries none of it.
"""
from __future__ import annotations

import argparse
import collections
import ctypes as C

import numpy as np
import torch

from . import binding as B
from . import build, synth

SLOTS = 1 << 18


def slot_of(key: int) -> int:
    return ((key * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF) >> 40 & (SLOTS - 1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama2-7b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--spec", action="store_true", help="one self-speculative step instead of one greedy token")
    ap.add_argument("--layers", default="4", help="layers whose launches are listed one by one")
    ap.add_argument("--prompt", type=int, default=0, help="prompt length (default: the workload's)")
    a = ap.parse_args()
    if not build.TRACE_LIB.exists():
        raise SystemExit("run `python -m paper_2404_16710_b200.build --trace` first")
    B.LIB_PATH = build.TRACE_LIB  # before the first call into the binding
    L = B.lib()
    L.ls_trace_reset.argtypes, L.ls_trace_read.argtypes = [C.c_int], [C.c_void_p]
    wl = synth.WORKLOADS[a.workload]
    s, E, d, P = wl.shape, wl.exit_layer, wl.num_draft, a.prompt or wl.n_prompt
    w = synth.make_weights(s, wl.weight_seed, E, wl.late_scale, device="cuda")
    max_seq = P + 64
    gm = B.Model(s, w, max_seq, 64, max(d, 1))
    B.ls_prefill(gm.h, synth.make_prompt(s.vocab, P, wl.prompt_seed))
    B.ls_decode(gm.h, 0, 0, 8)
    if a.spec:
        B.ls_decode(gm.h, E, d, 8)
    torch.cuda.synchronize()
    assert L.ls_trace_reset(1) == 0
    B.ls_decode(gm.h, E if a.spec else 0, d if a.spec else 0, 1)
    rec = np.zeros((SLOTS, 8), dtype=np.uint64)
    assert L.ls_trace_read(rec.ctypes.data) == 0
    L.ls_trace_reset(0)

    # keys: weight matrices, and each layer's K pages (the workspace starts with them)
    layer_kv_bytes = -(-max_seq // 64) * s.n_kv_heads * 64 * s.head_dim * 2
    names = {}
    for l in range(s.n_layers):
        for nm, key in (("qkv", w["wq"][l].data_ptr()), ("o", w["wo"][l].data_ptr()),
                        ("gate_up", w["w_gate"][l].data_ptr()), ("down", w["w_down"][l].data_ptr()),
                        ("attn", gm.workspace.data_ptr() + l * layer_kv_bytes)):
            for sub in (0, 1):
                names[key + sub] = f"L{l:02d}.{nm}" + (".M" if sub else "")
    for sub in (0, 1):
        names[w["lm_head"].data_ptr() + sub] = "lm_head" + (".M" if sub else "")
    taken = collections.Counter(slot_of(k) for k in names)
    shared = sorted(n for k, n in names.items() if taken[slot_of(k)] > 1)
    if shared:
        print("launches that share a trace slot (their records are merged):", ", ".join(shared))
    rows = sorted((int(r[1]), names.get(int(r[0]), hex(int(r[0]))), *[int(x) for x in r[1:8]]) for r in rec[rec[:, 7] > 0])
    t0 = rows[0][0]
    us = lambda t: (t - t0) / 1e3
    print(f"{len(rows)} launches recorded; {us(max(r[7] for r in rows)):.1f} us from the first CTA start to the last end")
    print("(.M: a pass of more than one row; with --spec the draft passes share the records of layers < E)")
    print(f"{'launch':16s}{'CTAs/8':>7s} | start first..last | wait released first..last | end first..last | prev end->end | prev end->release")
    shown = [int(x) for x in a.layers.split(",") if x]
    per_kind = collections.defaultdict(lambda: ([], [], []))
    prev_end = None
    for _, nm, s0, s1, w0, w1, e0, e1, n in rows:
        kind = nm.split(".", 1)[1] if nm.startswith("L") else nm
        if prev_end is not None:
            k = per_kind[kind]
            k[0].append((e1 - prev_end) / 1e3), k[1].append((w0 - prev_end) / 1e3), k[2].append((prev_end - s0) / 1e3)
            if any(nm.startswith(f"L{l:02d}.") for l in shown) or nm.startswith("lm_head"):
                print(f"{nm:16s}{n:7d} | {us(s0):8.2f} {us(s1):8.2f} | {us(w0):8.2f} {us(w1):8.2f} | {us(e0):8.2f} {us(e1):8.2f} |"
                      f" {(e1 - prev_end) / 1e3:7.2f} | {(w0 - prev_end) / 1e3:6.2f}")
        prev_end = e1
    print("medians over the pass (us):")
    for kind, (dur, gap, lead) in per_kind.items():
        print(f"  {kind:10s} launches {len(dur):3d}  prev end -> end {np.median(dur):6.2f}  prev end -> wait released "
              f"{np.median(gap):5.2f}  first CTA resident before prev end {np.median(lead):6.2f}")


if __name__ == "__main__":
    main()
