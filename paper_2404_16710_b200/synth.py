"""Seeded synthetic inputs: model shapes, weights and prompts.

This module holds NONE of the method's arithmetic.  It only draws random
tensors, so that the CUDA library and the CPU oracle can be given the very same
inputs.  The paper's own workloads (trained LayerSkip checkpoints of Llama-2
7B/13B and Llama-3 8B on summarisation / code / parsing prompts) are not
available offline; these inputs keep their shapes and regimes:

* matrices and the embedding table: N(0, 0.02), rounded once to bf16;
* norm gains: 1 + N(0, 0.02), rounded once to bf16 (so a wrong gain index shows);
* the residual output projections (o_proj, down_proj) of layers >= ``scale_from``
  are multiplied by ``late_scale`` before rounding: the smaller the factor, the
  closer the exit-layer prediction is to the full model's, which controls the
  draft acceptance rate;
* prompts: i.i.d. uniform token ids over the vocabulary.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np
import torch


@dataclass(frozen=True)
class Shape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 1e4

    def dict(self):
        return asdict(self)

    @property
    def layer_weight_bytes(self) -> int:
        qkv = (self.n_heads + 2 * self.n_kv_heads) * self.head_dim * self.d_model
        o = self.n_heads * self.head_dim * self.d_model
        return 2 * (qkv + o + 3 * self.d_model * self.d_ffn)

    @property
    def lm_head_bytes(self) -> int:
        return 2 * self.vocab * self.d_model

    @property
    def kv_bytes_per_token_layer(self) -> int:
        return 2 * 2 * self.n_kv_heads * self.head_dim


@dataclass(frozen=True)
class Workload:
    shape: Shape
    n_prompt: int
    max_new: int
    exit_layer: int
    num_draft: int
    late_scale: float
    weight_seed: int = 1234
    prompt_seed: int = 4321


TINY = Shape("tiny", 4, 256, 4, 4, 64, 688, 1024)
LLAMA2_7B = Shape("llama2-7b-shaped", 32, 4096, 32, 32, 128, 11008, 32000)
LLAMA2_13B = Shape("llama2-13b-shaped", 40, 5120, 40, 40, 128, 13824, 32000)
LLAMA3_8B = Shape("llama3-8b-shaped", 32, 4096, 32, 8, 128, 14336, 128256, rope_theta=5e5)
# small shapes for unit tests: grouped KV heads, ragged K (d_ffn not a multiple of 32)
MICRO_GQA = Shape("micro-gqa", 3, 64, 4, 2, 16, 88, 160)
MICRO_MHA = Shape("micro-mha", 3, 64, 4, 4, 16, 88, 160)
# small shape the CUDA kernels accept (head_dim 64), with grouped KV heads, a ragged K
# (d_ffn = 2*32 + 24) and a vocabulary that is not a multiple of the 16-row tile
GPU_MICRO = Shape("gpu-micro", 3, 96, 4, 2, 64, 88, 200)

WORKLOADS = {
    "tiny": Workload(TINY, 32, 64, 2, 3, 0.1),
    "llama2-7b": Workload(LLAMA2_7B, 1024, 256, 8, 6, 0.05),
    "llama2-13b": Workload(LLAMA2_13B, 1024, 256, 10, 8, 0.05),
    "llama3-8b": Workload(LLAMA3_8B, 512, 128, 8, 4, 0.05),
}
# the sweep on the 7B shape: prompt 4096, 256 new tokens
SWEEP_EXIT = (4, 8, 16)
SWEEP_DRAFT = (2, 4, 8, 12)
SWEEP_SCALE = (0.02, 0.05, 0.2)


def sweep_workload(exit_layer: int, num_draft: int, late_scale: float) -> Workload:
    return Workload(LLAMA2_7B, 4096, 256, exit_layer, num_draft, late_scale)


PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def _normal(shape, seed, device, scale, offset=0.0):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    t.mul_(scale)
    if offset:
        t.add_(offset)
    return t.to(torch.bfloat16)


def make_weights(shape: Shape, seed: int, scale_from: int, late_scale: float,
                 device: str = "cpu") -> dict:
    """bf16 torch tensors on ``device``; every tensor has a seed of its own, so a
    tensor's values do not depend on which other tensors were drawn."""
    s = shape
    qw, kvw = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    dims = {"wq": (qw, s.d_model), "wk": (kvw, s.d_model), "wv": (kvw, s.d_model),
            "wo": (s.d_model, qw), "w_gate": (s.d_ffn, s.d_model), "w_up": (s.d_ffn, s.d_model),
            "w_down": (s.d_model, s.d_ffn)}
    base = int(seed) * 100003
    w = {"tok_embed": _normal((s.vocab, s.d_model), base + 1, device, 0.02),
         "final_norm": _normal((s.d_model,), base + 2, device, 0.02, 1.0),
         "lm_head": _normal((s.vocab, s.d_model), base + 3, device, 0.02)}
    for name in PER_LAYER:
        w[name] = []
    for l in range(s.n_layers):
        for i, name in enumerate(PER_LAYER):
            sd = base + 1000 + 16 * l + i
            if name in ("attn_norm", "ffn_norm"):
                w[name].append(_normal((s.d_model,), sd, device, 0.02, 1.0))
            else:
                sc = 0.02
                if name in ("wo", "w_down") and l >= scale_from:
                    sc *= late_scale
                w[name].append(_normal(dims[name], sd, device, sc))
    return w


def amplify(weights: dict, factor: float) -> dict:
    """Scale every matrix (not the norm gains) by ``factor``: N(0, 0.02) draws on a narrow
    model give nearly flat logits, a louder draw makes comparisons sensitive to every term."""
    out = {}
    for k, v in weights.items():
        if k in ("attn_norm", "ffn_norm", "final_norm"):
            out[k] = v
        elif isinstance(v, list):
            out[k] = [(t.float() * factor).to(torch.bfloat16) for t in v]
        else:
            out[k] = (v.float() * factor).to(torch.bfloat16)
    return out


def make_prompt(vocab: int, n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(int(seed))
    return rng.integers(0, vocab, size=n, dtype=np.int32)


def as_uint16(weights: dict) -> dict:
    """The same weights as host numpy arrays of bf16 bit patterns."""
    def one(t):
        return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return {k: ([one(t) for t in v] if isinstance(v, list) else one(v)) for k, v in weights.items()}


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even), for hand-made test inputs."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_values(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64 values (exact)."""
    u = bits.astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)
