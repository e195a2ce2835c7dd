"""Shared helpers of the GPU parity tests: the same seeded inputs go to the CUDA library
(through its C ABI) and to the CPU oracle."""
import numpy as np
import torch

from oracle import ls_oracle as O
from paper_2404_16710_b200 import binding as B
from paper_2404_16710_b200 import synth

LOGIT_TOL = 3e-2  # max|delta| <= LOGIT_TOL * max|logit| (bf16 weights/activations, fp32 accumulation)


def make_pair(shape, seed, scale_from, late_scale, max_seq, page_size=64, max_draft=8, eos_id=-1,
              linear_path=B.LS_LINEAR_AUTO, amplify=None, oracle=True, draw_on="cuda"):
    """-> (gpu Model, oracle Model or None).  draw_on="cpu": the weights are drawn by the host
    generator (whose stream differs from the device's) and then moved to the GPU, for tests whose
    seeds were picked with the oracle alone on a machine without a GPU."""
    w = synth.make_weights(shape, seed, scale_from, late_scale, device=draw_on)
    if draw_on != "cuda":
        w = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}
    if amplify:
        w = synth.amplify(w, amplify)
    gm = B.Model(shape, w, max_seq, page_size, max_draft, eos_id, linear_path)
    om = None
    if oracle:
        cfg = O.Config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                       shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta, max_seq, eos_id)
        om = O.Model(cfg, synth.as_uint16(w))
    return gm, om


def assert_logits_close(gpu, ref, what=""):
    scale = np.abs(ref).max()
    err = np.abs(gpu.astype(np.float64) - ref).max()
    assert err <= LOGIT_TOL * scale, f"{what}: max|delta| {err:.4g} > {LOGIT_TOL} * max|logit| {scale:.4g}"
    return err / scale


def first_low_margin(margins, maxabs):
    """index of the first generated token whose oracle top-1/top-2 gap is within the tolerance"""
    low = np.nonzero(margins <= LOGIT_TOL * maxabs)[0]
    return int(low[0]) if low.size else len(margins)


def bf16_cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()


def bits(t):
    """torch bf16 tensor -> numpy uint16 bit patterns"""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def vals(t):
    """torch bf16 tensor -> float64 numpy values"""
    return t.detach().float().cpu().numpy().astype(np.float64)
