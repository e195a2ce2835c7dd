"""Time single kernels of the decode path on a workload's shapes, through the C ABI.

    python -m paper_2404_16710_b200.opbench --workload llama2-7b --layers 4 --ops gate_up_swiglu --rows 7

Each op is launched ``iters`` times (as one CUDA graph) with CUDA events around the batch,
rotating over the weights of ``layers`` layers so that no launch finds its weights in L2 (one 7B-shaped
gate+up pair is 180 MB, the L2 126 MB).  Algorithmic bytes of a launch are its weight
bytes (2 N K; the activations, M K 2 bytes, are noise).  Also the small driver to run
under a profiler: few launches, a few GB on the device.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B
from . import synth

OPS = ("gate_up_swiglu", "down_residual", "qkv_proj", "o_residual", "lm_head_argmax", "attention", "rmsnorm")


def time_op(fn, n_rot, iters=40, warm=5):
    """mean device time (ms) of one launch of fn: ``iters`` launches are captured into a
    CUDA graph (so that the host's launch rate does not bound kernels of a few
    microseconds) and the graph is replayed between two CUDA events on its stream."""
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        for i in range(warm):
            fn(i % n_rot)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for i in range(iters):
                fn((warm + i) % n_rot)
        g.replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        g.replay()
        e1.record(st)
        st.synchronize()
    torch.cuda.current_stream().wait_stream(st)
    return e0.elapsed_time(e1) / iters


def op_cases(shape, w, path, M, n_ctx=1030):
    """name -> (callable(layer index), algorithmic bytes per launch, number of distinct weights).
    attention: rows at positions n_ctx .. n_ctx+M-1 over a cache of n_ctx earlier tokens; its
    algorithmic bytes are the K and V rows it must read."""
    D, F, V = shape.d_model, shape.d_ffn, shape.vocab
    L = len(w["wq"])
    qw = shape.n_heads * shape.head_dim
    kvw = shape.n_kv_heads * shape.head_dim
    g = torch.Generator(device="cuda").manual_seed(7)
    h = torch.randn((M, D), device="cuda", generator=g).bfloat16()
    a = torch.randn((M, F), device="cuda", generator=g).bfloat16()
    o = torch.randn((M, qw), device="cuda", generator=g).bfloat16()
    x = torch.zeros((M, D), dtype=torch.float32, device="cuda")
    act = torch.empty((M, F), dtype=torch.bfloat16, device="cuda")
    qkv = torch.empty((M, qw + 2 * kvw), dtype=torch.float32, device="cuda")
    tok = torch.empty((M,), dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.ls_op_lm_head_scratch_bytes(V), dtype=torch.uint8, device="cuda")
    # q, k and v projections as one matrix of the fused launch's size
    wqkv = [torch.cat([w["wq"][i], w["wk"][i], w["wv"][i]]) for i in range(L)]
    heads = [w["lm_head"], w["tok_embed"]]
    # paged KV cache of a few layers (rotated over), identity page table
    Hq, Hkv, hd, ps = shape.n_heads, shape.n_kv_heads, shape.head_dim, 64
    max_seq = n_ctx + M + 1
    n_pages = -(-max_seq // ps)
    kvl = min(L, 8)
    kp = [torch.randn((n_pages, Hkv, ps, hd), device="cuda", generator=g).bfloat16() for _ in range(kvl)]
    vp = [torch.randn((n_pages, Hkv, ps, hd), device="cuda", generator=g).bfloat16() for _ in range(kvl)]
    table = torch.arange(n_pages, dtype=torch.int32, device="cuda")
    q = (torch.randn((M, qw), device="cuda", generator=g) * 0.3).bfloat16()
    ao = torch.empty((M, qw), dtype=torch.bfloat16, device="cuda")
    xs = torch.randn((M, D), device="cuda", generator=g)
    hn = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
    gain = w["attn_norm"][0]
    kv_bytes = 2 * 2 * Hkv * hd * (n_ctx + M)
    return {
        "attention": (lambda i: B.ls_op_attention(q, n_ctx, Hq, Hkv, hd, ps, table, max_seq, kp[i % kvl], vp[i % kvl], ao), kv_bytes, kvl),
        "rmsnorm": (lambda i: B.ls_op_rmsnorm(xs, gain, 1e-5, hn), 4 * M * D, 1),
        "gate_up_swiglu": (lambda i: B.ls_op_gate_up_swiglu(path, w["w_gate"][i % L], w["w_up"][i % L], h, act),
                           4 * F * D, L),
        "down_residual": (lambda i: B.ls_op_linear(path, w["w_down"][i % L], a, x, True), 2 * F * D, L),
        "qkv_proj": (lambda i: B.ls_op_linear(path, wqkv[i % L], h, qkv, False), 2 * (qw + 2 * kvw) * D, L),
        "o_residual": (lambda i: B.ls_op_linear(path, w["wo"][i % L], o, x, True), 2 * D * qw, L),
        "lm_head_argmax": (lambda i: B.ls_op_lm_head_argmax(path, heads[i % 2], h, scratch, tok), 2 * V * D, 2),
    }


PROMPT_OPS = ("prompt_gemm_qkv", "prompt_gemm_gate", "prompt_gemm_down", "prompt_attention")


def prompt_cases(shape, w, R):
    """Kernels of the prompt pass on R rows: name -> (callable(layer index), flops per launch, distinct weights).
    The GEMMs are the projections of one block of rows; attention is causal over the R rows themselves."""
    D, F = shape.d_model, shape.d_ffn
    L = len(w["wq"])
    Hq, Hkv, hd, ps = shape.n_heads, shape.n_kv_heads, shape.head_dim, 64
    qw, kvw = Hq * hd, Hkv * hd
    g = torch.Generator(device="cuda").manual_seed(11)
    h = torch.randn((R, D), device="cuda", generator=g).bfloat16()
    a = torch.randn((R, F), device="cuda", generator=g).bfloat16()
    wqkv = [torch.cat([w["wq"][i], w["wk"][i], w["wv"][i]]) for i in range(L)]
    cq = torch.empty((R, qw + 2 * kvw), dtype=torch.float32, device="cuda")
    cf = torch.empty((R, F), dtype=torch.float32, device="cuda")
    cd = torch.zeros((R, D), dtype=torch.float32, device="cuda")
    n_pages = -(-(R + 1) // ps)
    kp = torch.randn((n_pages, Hkv, ps, hd), device="cuda", generator=g).bfloat16()
    vp = torch.randn((n_pages, Hkv, ps, hd), device="cuda", generator=g).bfloat16()
    table = torch.arange(n_pages, dtype=torch.int32, device="cuda")
    q = (torch.randn((R, qw), device="cuda", generator=g) * 0.3).bfloat16()
    ao = torch.empty((R, qw), dtype=torch.bfloat16, device="cuda")
    return {
        "prompt_gemm_qkv": (lambda i: B.ls_op_gemm(h, wqkv[i % L], cq), 2 * R * (qw + 2 * kvw) * D, L),
        "prompt_gemm_gate": (lambda i: B.ls_op_gemm(h, w["w_gate"][i % L], cf), 2 * R * F * D, L),
        "prompt_gemm_down": (lambda i: B.ls_op_gemm(a, w["w_down"][i % L], cd, True), 2 * R * D * F, L),
        "prompt_attention": (lambda i: B.ls_op_prefill_attention(q, 0, Hq, Hkv, hd, ps, table, n_pages * ps, kp, vp, ao),
                             4 * Hq * hd * R * (R + 1) // 2, 1),
    }


def prompt_rates(shape, w, R, ops=PROMPT_OPS, iters=20, warm=3):
    out = {}
    cases = prompt_cases(shape, w, R)
    for name in ops:
        fn, flops, rot = cases[name]
        ms = time_op(fn, rot, iters, warm)
        out[f"{name}@R={R}"] = {"ms": round(ms, 5), "TFLOP/s": round(flops / ms / 1e9, 1), "flops": flops}
    return out


def kernel_rooflines(shape, w, path, rows, peak_gbs, ops=OPS, iters=40, warm=5, chained=True):
    """Per op and pass size: one launch alone (launches serialised: each starts when the one before
    has drained) and, with ``chained``, the same launches linked by programmatic dependent launch as
    inside the decode loop (``ms_chained``: a launch's CTAs move in and prefetch while its
    predecessor's last CTAs finish).  Fractions are algorithmic bytes / time / peak_gbs."""
    out = {}
    for M in rows:
        cases = op_cases(shape, w, path, M)
        for name in ops:
            fn, nbytes, rot = cases[name]
            ms = time_op(fn, rot, iters, warm)
            e = {"ms": round(ms, 5), "GB/s": round(nbytes / ms / 1e6, 1),
                 "frac": round(nbytes / ms / 1e6 / peak_gbs, 4), "bytes": nbytes}
            if chained:
                B.ls_op_chain(True)
                try:
                    msc = time_op(fn, rot, iters, warm)
                finally:
                    B.ls_op_chain(False)
                e["ms_chained"] = round(msc, 5)
                e["frac_chained"] = round(nbytes / msc / 1e6 / peak_gbs, 4)
            out[f"{name}@M={M}"] = e
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama2-7b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=4, help="layers of weights to create and rotate over")
    ap.add_argument("--ops", default=",".join(OPS))
    ap.add_argument("--rows", default="1,7")
    ap.add_argument("--path", default="mma", choices=["fma", "mma"])
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--warm", type=int, default=5)
    ap.add_argument("--peak", type=float, default=6553.9, help="GB/s the fractions are quoted against")
    ap.add_argument("--prompt-rows", type=int, default=0, metavar="R",
                    help="instead: the prompt pass's GEMMs and attention on R rows (TFLOP/s); --ops picks among "
                         + ", ".join(PROMPT_OPS))
    a = ap.parse_args()
    from dataclasses import replace
    wl = synth.WORKLOADS[a.workload]
    shape = replace(wl.shape, n_layers=a.layers)
    w = synth.make_weights(shape, wl.weight_seed, wl.exit_layer, wl.late_scale, device="cuda")
    path = B.LS_LINEAR_MMA if a.path == "mma" else B.LS_LINEAR_FMA
    if a.prompt_rows:
        ops = [o for o in a.ops.split(",") if o in PROMPT_OPS] or list(PROMPT_OPS)
        res = prompt_rates(shape, w, a.prompt_rows, ops, a.iters, a.warm)
        for k, v in res.items():
            print(f"{k:28s} {v['ms'] * 1e3:8.2f} us  {v['TFLOP/s']:8.1f} TFLOP/s")
        print(json.dumps(res))
        return
    res = kernel_rooflines(shape, w, path, [int(r) for r in a.rows.split(",")], a.peak,
                           [o for o in a.ops.split(",") if o], a.iters, a.warm)
    for k, v in res.items():
        print(f"{k:28s} {v['ms'] * 1e3:8.2f} us  {v['GB/s']:8.1f} GB/s  {v['frac']:.3f} of {a.peak:.0f}   chained "
              f"{v['ms_chained'] * 1e3:8.2f} us  {v['frac_chained']:.3f}")
    print(json.dumps(res))


if __name__ == "__main__":
    main()
