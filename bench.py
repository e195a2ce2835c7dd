#!/usr/bin/env python
"""Benchmark of the batch-1 self-speculative greedy decode loop (LayerSkip Sec. 4.3).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama2-7b] [--impl reference]

One "step" is one run of the whole decode loop (draft, verify, accept until max_new
tokens exist) from a prefilled prompt.  The metric is generated tokens per second of
self-speculative decoding; the same library's full-model greedy tokens/s, the effective
HBM bandwidth of the schedule, the dominant kernel's roofline and the CPU oracle's speed
on a bounded sample are reported beside it.  Inputs are seeded and synthetic (see
paper_2404_16710_b200/synth.py); weights (13 GB on the Llama-2-7B shape) are far larger
than the 126 MB L2, so consecutive timed iterations cannot hit in cache.

With N > 1 (torchrun) every rank runs an independent replica on its own GPU: the decode
loop of one sequence is a single dependency chain and does not shard; no collective
touches the data path.  `--impl reference` times the CPU oracle on host cores (rank 0
only).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2404_16710_b200 import synth  # noqa: E402

METRIC = "batch-1 generated tokens/s, self-speculative greedy decode"
UNIT = "tokens/s"

# thresholds on the exit-logit margin tried by the adaptive-draft-length leg (logit units)
ADAPTIVE_MARGINS = (0.02, 0.05, 0.1, 0.2, 0.4)
# DRAM bytes (read + write) per launch, as ncu counted them, are kept beside the ncu summaries:
# the table in this file has one row per (workload, op, rows) that was captured.
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.md")


def measured_traffic(workload, op, rows):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch from the committed ncu table, or
    None when that (workload, op, rows) has no row there."""
    try:
        with open(TRAFFIC_TABLE) as f:
            for line in f:
                c = [x.strip() for x in line.strip().strip("|").split("|")]
                if len(c) >= 5 and c[0] == workload and c[1] == op and c[2] == str(rows):
                    return float(c[3]) + float(c[4])
    except OSError:
        pass
    return None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *a):
        self.summary = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if not self.proc:
            return
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if sm:
            self.summary = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                            "samples": len(sm)}


def max_over_ranks(value, dist, device):
    """The slowest rank's time: replicas are independent, the job ends when the last one does."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(world, steps, new_tokens, total_ms):
    """Whole-job throughput of `world` independent replicas timed by the slowest one."""
    return world * steps * new_tokens / (total_ms / 1e3)


def oracle_model(wl, weights, max_seq):
    from oracle import ls_oracle as O
    s = wl.shape
    cfg = O.Config(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab,
                   s.rms_eps, s.rope_theta, max_seq)
    return O, O.Model(cfg, synth.as_uint16(weights))


def cpu_sample(wl, om, O, prompt, n_prompt, max_new):
    """The oracle as it stands on a bounded sample of the workload -> (tokens/s, description)."""
    t0 = time.perf_counter()
    ids, acc, _ = om.generate_spec(prompt[:n_prompt], wl.exit_layer, wl.num_draft, max_new)
    dt = time.perf_counter() - t0
    desc = (f"{wl.shape.name}: prompt truncated to its first {n_prompt} ids (prefill of {n_prompt - 1} tokens "
            f"included in the time), {len(ids)} new tokens, E={wl.exit_layer}, d={wl.num_draft}, "
            f"{len(acc)} steps, {dt:.1f} s")
    return len(ids) / dt, desc


def cpu_sample_sizes(shape):
    # about 10-30 s of oracle work: ~1 s per token-pass on the 7B shape with 8 cores
    big = shape.n_layers * shape.layer_weight_bytes > 2e9
    return (3, 5) if big else (16, 32)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.WORKLOADS[args.workload]
    dev = "cuda" if torch.cuda.is_available() else "cpu"  # input generation only
    w = synth.make_weights(wl.shape, wl.weight_seed, wl.exit_layer, wl.late_scale, device=dev)
    n_prompt, max_new = cpu_sample_sizes(wl.shape)
    O, om = oracle_model(wl, w, n_prompt + max_new + wl.num_draft + 2)
    del w
    prompt = synth.make_prompt(wl.shape.vocab, wl.n_prompt, wl.prompt_seed)
    steps = max(1, min(args.steps, 3))
    vals, desc = [], ""
    for i in range(min(args.warmup, 1) + steps):
        v, desc = cpu_sample(wl, om, O, prompt, n_prompt, max_new)
        if i >= min(args.warmup, 1):
            vals.append(v)
    value = float(np.mean(vals))
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * max_new / value,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": args.workload, "shape": wl.shape.name, "n_prompt": n_prompt,
                      "max_new": max_new, "exit_layer": wl.exit_layer, "num_draft": wl.num_draft,
                      "late_scale": wl.late_scale,
                      "note": f"CPU oracle (fp64, OpenMP) on a bounded sample: the workload's prompt cut to its first "
                              f"{n_prompt} ids and {max_new} new tokens (the workload itself: prompt {wl.n_prompt}, "
                              f"{wl.max_new} new tokens)"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": desc},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def run_own(args):
    from paper_2404_16710_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = synth.WORKLOADS[args.workload]
    s = wl.shape
    E, d, P, NEW = wl.exit_layer, wl.num_draft, wl.n_prompt, wl.max_new
    peak, peak_kind = peaks()

    if args.profile_prompt:
        P = args.profile_prompt
    w = synth.make_weights(s, wl.weight_seed, E, wl.late_scale, device="cuda")
    max_seq = P + NEW + d + 1
    gm = B.Model(s, w, max_seq, 64, max(d, 1))
    prompt = synth.make_prompt(s.vocab, P, wl.prompt_seed + rank)
    path = B.LS_LINEAR_MMA if d + 1 > 4 else B.LS_LINEAR_FMA

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    if args.profile_prompt:
        for _ in range(max(1, args.warmup)):
            B.ls_prefill(gm.h, prompt)
        torch.cuda.synchronize()
        torch.cuda.profiler.start()
        B.ls_prefill(gm.h, prompt)
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()
        print(json.dumps({"profile_prompt": P, "prefill_ms": round(gm.stats().prefill_ms, 2)}))
        return
    if args.profile_region:
        B.ls_prefill(gm.h, prompt)
        for _ in range(max(1, args.warmup)):
            B.ls_decode(gm.h, E, d, args.profile_region)
            B.ls_decode(gm.h, 0, 0, args.profile_region)
        torch.cuda.synchronize()
        torch.cuda.profiler.start()
        B.ls_decode(gm.h, E, d, args.profile_region)
        B.ls_decode(gm.h, 0, 0, args.profile_region)
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()
        print(json.dumps({"profile_region": args.profile_region, "launches": int(gm.stats().kernel_launches)}))
        return

    # ---- device-resident timing: prompts already prefilled in HBM, decode loop only.  The timed steps
    # rotate over a few prompts of the same recipe (each on a handle of its own, prefilled beforehand):
    # the accepted drafts per step of a synthetic model hinge on near-ties of its exit logits and
    # swing by +-0.4 from one prompt to the next, so one prompt repeated K times would put that draw
    # into the headline number; full greedy decoding runs over the same prompts.
    n_prompts = max(1, min(args.steps, 4))
    prompts = [prompt] + [synth.make_prompt(s.vocab, P, wl.prompt_seed + rank + 7919 * i) for i in range(1, n_prompts)]
    gms = [gm] + [B.Model(s, w, max_seq, 64, max(d, 1)) for _ in range(1, n_prompts)]
    prefill_all = []
    for g, pr in zip(gms, prompts):
        B.ls_prefill(g.h, pr)
        prefill_all.append(g.stats().prefill_ms)
    prefill_ms = statistics.median(prefill_all)
    for _ in range(args.warmup):
        B.ls_decode(gm.h, E, d, NEW)
    spec_out = []
    for g in gms:
        B.ls_decode(g.h, E, d, NEW)
        spec_out.append(B.ls_read_output(g.h, NEW))
    spec_ids = spec_out[0][0]
    acc = np.concatenate([a for _, a in spec_out])
    launches = 0
    loop_ms, loop_bytes = [], []
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clk:
        e0.record()
        for k in range(args.steps):
            g = gms[k % n_prompts]
            B.ls_decode(g.h, E, d, NEW)
            st = g.stats()
            launches += st.kernel_launches
            loop_ms.append(st.decode_ms)
            loop_bytes.append(st.weight_bytes + st.kv_bytes)
        e1.record()
        barrier()
    total_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
    st = gm.stats()
    value = job_tokens_per_s(world, args.steps, NEW, total_ms)
    sched_bytes = statistics.mean(loop_bytes)
    loop_gbs = sum(loop_bytes) / (sum(loop_ms) / 1e3) / 1e9
    spec_ms_per_step = sum(loop_ms) / sum(len(spec_out[k % n_prompts][1]) for k in range(args.steps))

    # ---- end to end through the public call: host prompt in, host ids out, prefill included.  Taken right
    # after the timed region, in the same power and clock state (the later legs run hotter).
    e2e_ms = []
    for i in range(1 + max(1, min(args.steps, 4))):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ids, a2 = gm.generate(prompts[i % n_prompts], E, d, NEW)
        if i:
            e2e_ms.append((time.perf_counter() - t0) * 1e3)
    e2e_worst = max_over_ranks(statistics.mean(e2e_ms), dist, "cuda")  # mean call over the rotated prompts, slowest rank
    est = gm.stats()
    e2e = {"value": world * NEW / (e2e_worst / 1e3), "unit": UNIT, "h2d_bytes_per_step": 4 * P + 32 * 2,
           "d2h_bytes_per_step": 4 * len(ids) + 4 * len(a2) + 32 * (est.host_syncs + 1),
           "includes": "prompt H2D, prefill of the prompt, decode loop, ids D2H", "prefill_ms": est.prefill_ms}
    B.ls_prefill(gm.h, prompts[0])  # the later legs start from the first prompt's cache again

    # ---- the same library's full-model greedy decoding, same model, same prompts
    for _ in range(min(args.warmup, 2)):
        B.ls_decode(gm.h, 0, 0, NEW)
    full_ms, full_bytes, lossless = [], [], True
    for g, (ids_g, _) in zip(gms, spec_out):
        B.ls_decode(g.h, 0, 0, NEW)
        fst = g.stats()
        full_ms.append(fst.decode_ms)
        full_bytes.append(fst.weight_bytes + fst.kv_bytes)
        lossless = lossless and bool(np.array_equal(B.ls_read_output(g.h, NEW)[0], ids_g))
    full_tok_s = NEW * len(full_ms) / (sum(full_ms) / 1e3)
    full_gbs = sum(full_bytes) / (sum(full_ms) / 1e3) / 1e9
    for g in gms[1:]:
        g.close()
    del gms

    # ---- the paper's "without KVQ reuse" ablation (Table 7): verify recomputes the early layers
    B.ls_decode_flags(gm.h, E, d, NEW, B.LS_DECODE_NO_EXIT_CACHE)
    B.ls_decode_flags(gm.h, E, d, NEW, B.LS_DECODE_NO_EXIT_CACHE)
    nst = gm.stats()
    no_reuse_ids, _ = B.ls_read_output(gm.h, NEW)
    no_reuse = {"value": NEW / (nst.decode_ms / 1e3), "unit": UNIT,
                "ids_equal": bool(np.array_equal(no_reuse_ids, spec_ids))}

    # ---- adaptive draft length (an extension beyond the paper's fixed d): drafting stops when the
    # exit-logit top-1/top-2 margin falls below a threshold; ids must not change
    adaptive = {"unit": UNIT, "max_draft": d, "points": []}
    for tau in ADAPTIVE_MARGINS:
        B.ls_decode_adaptive(gm.h, E, d, tau, NEW)
        B.ls_decode_adaptive(gm.h, E, d, tau, NEW)
        ast = gm.stats()
        a_ids, a_acc = B.ls_read_output(gm.h, NEW)
        a_dr = B.ls_read_drafted(gm.h, NEW)
        adaptive["points"].append({"min_margin": tau, "value": round(NEW / (ast.decode_ms / 1e3), 1),
                                   "kept_per_step": round(float(a_dr.mean()), 3),
                                   "accepted_per_step": round(float(a_acc.mean()), 3), "steps": int(len(a_acc)),
                                   "hbm_frac_measured": round((ast.weight_bytes + ast.kv_bytes) /
                                                              (ast.decode_ms / 1e3) / 1e9 / peak, 4),
                                   "ids_equal": bool(np.array_equal(a_ids, spec_ids))})
    adaptive["best"] = max(adaptive["points"], key=lambda p: p["value"])

    # ---- several sequences per pass (an extension; Sec. 9 of the paper leaves batching open): B
    # sequences share every pass, so each weight byte read serves all of them; aggregate tokens/s
    batch = {"unit": UNIT, "note": "B sequences x (d+1) rows <= 16 rows per pass; value = B * max_new / loop time; "
                                   "ids of every sequence checked against its own single-sequence greedy run",
             "points": []}
    if not args.no_batch:
        cap = -(-(P + NEW + d + 2) // 64) * 64
        for nb, bd in ((2, d), (4, 3), (8, 1), (2, 0), (4, 0), (8, 0)):
            if nb * (bd + 1) > 16 or nb * cap > 16384 or (bd and bd > d):
                continue
            gb = B.Model(s, w, nb * cap, 64, max(d, 1))
            prompts = [synth.make_prompt(s.vocab, P, wl.prompt_seed + 100 * rank + b) for b in range(nb)]
            B.ls_prefill_batch(gb.h, prompts)
            bE = E if bd else 0
            B.ls_decode_batch(gb.h, bE, bd, NEW)
            B.ls_decode_batch(gb.h, bE, bd, NEW)
            bst = gb.stats()
            outs = [B.ls_read_output_seq(gb.h, b, NEW) for b in range(nb)]
            equal = all(np.array_equal(outs[b][0], gb.generate_full(prompts[b], NEW)) for b in range(min(nb, 2)))
            batch["points"].append({
                "sequences": nb, "num_draft": bd, "rows_per_verify_pass": nb * (bd + 1),
                "value": round(nb * NEW / (bst.decode_ms / 1e3), 1), "per_sequence": round(NEW / (bst.decode_ms / 1e3), 1),
                "accepted_per_step": round(float(np.mean([o[1].mean() for o in outs])), 3) if bd else 0.0,
                "hbm_frac_measured": round((bst.weight_bytes + bst.kv_bytes) / (bst.decode_ms / 1e3) / 1e9 / peak, 4),
                "ids_equal_single_sequence_greedy": bool(equal)})
            gb.close()
            del gb
            torch.cuda.empty_cache()
        if batch["points"]:
            batch["best"] = max(batch["points"], key=lambda q: q["value"])

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": args.workload, "shape": s.name, "n_prompt": P, "max_new": NEW, "exit_layer": E,
                      "num_draft": d, "late_scale": wl.late_scale, "linear_path": "mma" if path == 2 else "fma",
                      "l2": "inputs (weights) larger than L2", "replicas": world, "prompts_rotated": n_prompts,
                      "timed_region": "decode loop from a prefilled prompt, device-resident",
                      "kernels_per_layer": 5, "prompt_pass": "persistent tcgen05 cta_group::2 GEMM, 256x256 tiles on CTA pairs, two TMEM accumulators, blocks of 1024 rows"},
           "e2e": e2e, "gpu_launches": int(launches), "clocks": clk.summary,
           # the numbers the value is read against come first, the long tables last
           "full_greedy": {"value": full_tok_s, "unit": UNIT, "hbm_GB/s": round(full_gbs, 1),
                           "hbm_frac_measured": round(full_gbs / peak, 4), "hbm_frac_8TBs": round(full_gbs / 8000, 4)},
           "speedup_vs_full_greedy": value / world / full_tok_s,
           "loop_hbm": {"GB/s": round(loop_gbs, 1), "frac_measured": round(loop_gbs / peak, 4),
                        "frac_8TBs": round(loop_gbs / 8000, 4), "bytes_per_loop": int(sched_bytes)},
           "ids_equal_full_greedy": lossless,
           "accepted_per_step": float(acc.mean()), "acceptance_rate": float(acc.mean() / d),
           "emitted_per_step": float(NEW * n_prompts / len(acc)), "spec_steps_per_prompt": [int(len(a)) for _, a in spec_out],
           "ms_per_spec_step": round(spec_ms_per_step, 4), "host_syncs": int(st.host_syncs),
           "prefill_ms": prefill_ms}

    if rank == 0 and world == 1:
        from paper_2404_16710_b200 import opbench
        ks = opbench.kernel_rooflines(s, w, path, (1, d + 1), peak)
        # The gate-up + SwiGLU linear is the largest kernel of a layer.  By share of the loop's time
        # its single-row launches (draft passes) dominate, its (d+1)-row launch (verify pass) is the
        # slower of the two per byte: the roofline object is the former, `verify_pass` the latter.
        fam = "mma" if path == 2 else "fma"

        def roof(M):
            k = ks[f"gate_up_swiglu@M={M}"]
            return {"rows": M, "achieved": k["GB/s"], "frac": k["frac"], "us_per_launch": round(k["ms"] * 1e3, 2),
                    "algorithmic_bytes": k["bytes"], "traffic": measured_traffic(args.workload, "gate_up_swiglu", M),
                    "frac_chained": k.get("frac_chained")}
        n_draft_launches = len(acc) / n_prompts * (d + 1) * E
        n_verify_launches = len(acc) / n_prompts * (s.n_layers - E)
        loop_ms_mean = statistics.mean(loop_ms)
        r1, rv = roof(1), roof(d + 1)
        out["roofline"] = {"bound": "hbm", "kernel": f"linear_{fam}_kernel, gate-up + SwiGLU, 1 row (draft passes)",
                           "achieved": r1["achieved"], "peak": peak, "unit": "GB/s", "frac": r1["frac"],
                           "traffic": r1["traffic"], "algorithmic_bytes": r1["algorithmic_bytes"],
                           "us_per_launch": r1["us_per_launch"], "frac_chained": r1["frac_chained"],
                           "share_of_loop_time_est": round(n_draft_launches * r1["us_per_launch"] / 1e3 / loop_ms_mean, 3),
                           "verify_pass": dict(rv, share_of_loop_time_est=round(
                               n_verify_launches * rv["us_per_launch"] / 1e3 / loop_ms_mean, 3)),
                           "peak_kind": f"of {peak_kind} (burst copy)",
                           "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch, "
                                             "profiles/dram_traffic_per_launch.md (null: not captured for this workload)",
                           "how": "CUDA events around a CUDA graph of 40 launches through the C ABI, rotating over the "
                                  "layers' weights (each launch streams from HBM), launches serialised (no dependent-launch "
                                  "overlap); frac_chained: the same launches linked by programmatic dependent launch, as "
                                  "inside the loop (ls_op_chain)"}
        # the CPU oracle on a bounded sample of the same workload
        n_p, n_new = cpu_sample_sizes(s)
        O, om = oracle_model(wl, w, n_p + n_new + d + 2)
        v, desc = cpu_sample(wl, om, O, prompt, n_p, n_new)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": desc}
        out["without_exit_cache_reuse"] = no_reuse
        out["batch"] = batch
        out["adaptive_draft"] = adaptive
        out["kernels"] = ks
    else:
        out["without_exit_cache_reuse"] = no_reuse
        out["batch"] = batch
        out["adaptive_draft"] = adaptive
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args):
    """The sweep on the Llama-2-7B shape (prompt 4096, 256 new tokens): exit layer x number of
    drafts x late-layer scale.  One JSON line per point, full-greedy numbers of the same model
    beside it.  Not the benchmark line: a table for the report."""
    from paper_2404_16710_b200 import binding as B
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    peak, _ = peaks()
    exits = [int(x) for x in args.sweep_exit.split(",")]
    drafts = [int(x) for x in args.sweep_draft.split(",")]
    scales = [float(x) for x in args.sweep_scale.split(",")]
    points = []
    for scale in scales:
        for E in exits:
            wl = synth.sweep_workload(E, max(drafts), scale)
            s, P, NEW = wl.shape, wl.n_prompt, wl.max_new
            w = synth.make_weights(s, wl.weight_seed, E, scale, device="cuda")
            gm = B.Model(s, w, P + NEW + max(drafts) + 1, 64, max(drafts))
            prompt = synth.make_prompt(s.vocab, P, wl.prompt_seed)
            B.ls_prefill(gm.h, prompt)
            prefill_ms = gm.stats().prefill_ms
            for _ in range(2):
                B.ls_decode(gm.h, 0, 0, NEW)
            fst = gm.stats()
            full_ids, _ = B.ls_read_output(gm.h, NEW)
            full_tok_s = NEW / (fst.decode_ms / 1e3)
            full_frac = (fst.weight_bytes + fst.kv_bytes) / (fst.decode_ms / 1e3) / 1e9 / peak
            for d in drafts:
                for _ in range(2):
                    B.ls_decode(gm.h, E, d, NEW)
                st = gm.stats()
                ids, acc = B.ls_read_output(gm.h, NEW)
                tok_s = NEW / (st.decode_ms / 1e3)
                points.append({
                    "sweep": "llama2-7b-shaped", "n_prompt": P, "max_new": NEW, "late_scale": scale, "exit_layer": E,
                    "num_draft": d, "tokens_per_s": round(tok_s, 1), "full_greedy_tokens_per_s": round(full_tok_s, 1),
                    "speedup": round(tok_s / full_tok_s, 3), "accepted_per_step": round(float(acc.mean()), 3),
                    "acceptance_rate": round(float(acc.mean() / d), 3),
                    "hbm_frac_measured": round((st.weight_bytes + st.kv_bytes) / (st.decode_ms / 1e3) / 1e9 / peak, 3),
                    "full_greedy_hbm_frac_measured": round(full_frac, 3),
                    "ids_equal_full_greedy": bool(np.array_equal(ids, full_ids)), "prefill_ms": round(prefill_ms, 1),
                    "host_syncs": int(st.host_syncs)})
                print(json.dumps(points[-1]), flush=True)
            gm.close()
            del gm, w
            torch.cuda.empty_cache()
    best = max(points, key=lambda p: p["tokens_per_s"])
    fracs = [p["hbm_frac_measured"] for p in points]
    fulls = [p["full_greedy_tokens_per_s"] for p in points]
    print(json.dumps({"sweep_summary": {
        "points": len(points), "all_ids_equal_full_greedy": all(p["ids_equal_full_greedy"] for p in points),
        "best": {k: best[k] for k in ("late_scale", "exit_layer", "num_draft", "tokens_per_s", "speedup",
                                      "accepted_per_step", "hbm_frac_measured")},
        "worst_speedup": min(p["speedup"] for p in points),
        "full_greedy_tokens_per_s": [min(fulls), max(fulls)],
        "full_greedy_hbm_frac_measured": [min(p["full_greedy_hbm_frac_measured"] for p in points),
                                          max(p["full_greedy_hbm_frac_measured"] for p in points)],
        "hbm_frac_measured": [min(fracs), max(fracs)]}}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="llama2-7b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--profile-region", type=int, default=0, metavar="NEW",
                    help="instead of the benchmark: prefill, warm up, then run one self-speculative and one "
                         "full-greedy decode of NEW tokens between cudaProfilerStart/Stop (for a profiler "
                         "started with --profile-from-start off) and exit")
    ap.add_argument("--profile-prompt", type=int, default=0, metavar="P",
                    help="instead of the benchmark: the prompt pass of a P-token prompt, warmed up, once between "
                         "cudaProfilerStart/Stop, then exit")
    ap.add_argument("--no-batch", action="store_true", help="skip the several-sequences-per-pass leg")
    ap.add_argument("--sweep", action="store_true", help="run the (exit layer, drafts, late scale) sweep instead")
    ap.add_argument("--sweep-exit", default=",".join(map(str, synth.SWEEP_EXIT)))
    ap.add_argument("--sweep-draft", default=",".join(map(str, synth.SWEEP_DRAFT)))
    ap.add_argument("--sweep-scale", default=",".join(map(str, synth.SWEEP_SCALE)))
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_own(args)


if __name__ == "__main__":
    main()
