"""ctypes front end of the CPU oracle (``ls_oracle.c``) -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares nothing with the CUDA library: its own C file, its own shared
object, its own argument marshalling.

Weights are handed over as numpy ``uint16`` arrays holding bf16 bit patterns
(row-major ``[out, in]``); all results are float64 / int32 numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ls_oracle.c"
_LIB = _HERE / "libls_oracle.so"


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fast-math: the summation order is the source's)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
               "-ffp-contract=off", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                 "max_seq", "eos_id")] + [("rms_eps", C.c_double), ("rope_theta", C.c_double)]


_U16P = C.POINTER(C.c_uint16)
_PP = C.POINTER(_U16P)


class _Wts(C.Structure):
    _fields_ = [("tok_embed", _U16P), ("final_norm", _U16P), ("lm_head", _U16P)] + \
               [(n, _PP) for n in ("attn_norm", "wq", "wk", "wv", "wo",
                                   "ffn_norm", "w_gate", "w_up", "w_down")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(str(build()))
        dp, ip = C.POINTER(C.c_double), C.POINTER(C.c_int32)
        i32 = C.c_int32
        L.lso_rmsnorm.argtypes = [dp, _U16P, i32, C.c_double, dp]
        L.lso_rope.argtypes = [dp, i32, i32, C.c_double]
        L.lso_linear.argtypes = [_U16P, i32, i32, dp, dp]
        L.lso_softmax.argtypes = [dp, i32]
        L.lso_silu.argtypes = [C.c_double]
        L.lso_silu.restype = C.c_double
        L.lso_attention.argtypes = [dp, dp, dp, i32, i32, i32, i32, dp]
        L.lso_argmax.argtypes = [dp, i32, dp, dp]
        L.lso_argmax.restype = i32
        L.lso_match.argtypes = [ip, ip, i32]
        L.lso_match.restype = i32
        L.lso_model_create.argtypes = [C.POINTER(_Cfg), C.POINTER(_Wts)]
        L.lso_model_create.restype = C.c_void_p
        L.lso_model_free.argtypes = [C.c_void_p]
        L.lso_teacher_logits.argtypes = [C.c_void_p, ip, i32, i32, dp, dp]
        L.lso_teacher_logits.restype = i32
        L.lso_teacher_logits_tail.argtypes = [C.c_void_p, ip, i32, i32, i32, dp, dp]
        L.lso_teacher_logits_tail.restype = i32
        L.lso_generate_full.argtypes = [C.c_void_p, ip, i32, i32, ip, ip, dp, dp]
        L.lso_generate_full.restype = i32
        L.lso_generate_early.argtypes = [C.c_void_p, ip, i32, i32, i32, ip, ip]
        L.lso_generate_early.restype = i32
        L.lso_generate_spec.argtypes = [C.c_void_p, ip, i32, i32, i32, i32, ip, ip, ip, ip, ip]
        L.lso_generate_spec.restype = i32
        L.lso_generate_adaptive.argtypes = [C.c_void_p, ip, i32, i32, i32, C.c_double, i32, ip, ip, ip, ip, ip,
                                            C.POINTER(C.c_double)]
        L.lso_generate_adaptive.restype = i32
        L.lso_num_threads.restype = i32
        _lib = L
    return _lib


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _u16(a):
    assert a.dtype == np.uint16 and a.flags.c_contiguous
    return a.ctypes.data_as(_U16P)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


# ---------------------------------------------------------------- elementary ops
def rmsnorm(x, g_bf16, eps):
    x = _f64(x)
    y = np.empty_like(x)
    lib().lso_rmsnorm(_dp(x), _u16(g_bf16), x.size, eps, _dp(y))
    return y


def rope(v, pos, theta):
    v = _f64(v).copy()
    lib().lso_rope(_dp(v), v.size, int(pos), float(theta))
    return v


def linear(w_bf16, h):
    n, k = w_bf16.shape
    h = _f64(h)
    assert h.size == k
    y = np.empty(n, dtype=np.float64)
    lib().lso_linear(_u16(w_bf16), n, k, _dp(h), _dp(y))
    return y


def softmax(s):
    s = _f64(s).copy()
    lib().lso_softmax(_dp(s), s.size)
    return s


def silu(z):
    return lib().lso_silu(float(z))


def attention(q, k, v, n_heads, n_kv_heads, head_dim):
    """q [Hq*hd]; k, v [n_keys, Hkv*hd] -> o [Hq*hd]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    o = np.empty(n_heads * head_dim, dtype=np.float64)
    lib().lso_attention(_dp(q), _dp(k), _dp(v), k.shape[0], n_heads, n_kv_heads, head_dim, _dp(o))
    return o


def argmax(z):
    z = _f64(z)
    mg, ma = C.c_double(), C.c_double()
    i = lib().lso_argmax(_dp(z), z.size, C.byref(mg), C.byref(ma))
    return i, mg.value, ma.value


def match(draft, verified):
    d = np.ascontiguousarray(draft, dtype=np.int32)
    v = np.ascontiguousarray(verified, dtype=np.int32)
    return lib().lso_match(_ip(d), _ip(v), d.size)


def num_threads() -> int:
    return lib().lso_num_threads()


# ---------------------------------------------------------------- the model
@dataclass
class Config:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 1e4
    max_seq: int = 256
    eos_id: int = -1


_PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class Model:
    """weights: dict with 'tok_embed', 'final_norm', 'lm_head' (uint16 arrays) and the
    per-layer names above (lists of uint16 arrays)."""

    def __init__(self, cfg: Config, weights: dict):
        self.cfg = cfg
        self._keep = weights  # the C side borrows the buffers
        c = _Cfg(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim,
                 cfg.d_ffn, cfg.vocab, cfg.max_seq, cfg.eos_id, cfg.rms_eps, cfg.rope_theta)
        w = _Wts()
        w.tok_embed, w.final_norm, w.lm_head = (_u16(weights[k]) for k in
                                                 ("tok_embed", "final_norm", "lm_head"))
        self._arrs = []
        for name in _PER_LAYER:
            assert len(weights[name]) == cfg.n_layers
            arr = (_U16P * cfg.n_layers)(*[_u16(a) for a in weights[name]])
            self._arrs.append(arr)
            setattr(w, name, C.cast(arr, _PP))
        self._h = lib().lso_model_create(C.byref(c), C.byref(w))
        if not self._h:
            raise RuntimeError("lso_model_create failed")

    def close(self):
        if self._h:
            lib().lso_model_free(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def teacher_logits(self, ids, exit_layer, want_exit=True, want_final=True):
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        n, V = ids.size, self.cfg.vocab
        ex = np.empty((n, V)) if want_exit else None
        fi = np.empty((n, V)) if want_final else None
        rc = lib().lso_teacher_logits(self._h, _ip(ids), n, exit_layer,
                                      _dp(ex) if want_exit else None,
                                      _dp(fi) if want_final else None)
        if rc:
            raise ValueError("lso_teacher_logits: bad arguments")
        return ex, fi

    def teacher_logits_tail(self, ids, exit_layer, first, want_exit=True, want_final=True):
        """Teacher-forced logits of positions first .. len(ids)-1 only ([len(ids) - first, V]); the
        earlier positions still run through every layer (they fill the cache)."""
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        n, V = ids.size, self.cfg.vocab
        ex = np.empty((n - first, V)) if want_exit else None
        fi = np.empty((n - first, V)) if want_final else None
        rc = lib().lso_teacher_logits_tail(self._h, _ip(ids), n, exit_layer, first,
                                           _dp(ex) if want_exit else None,
                                           _dp(fi) if want_final else None)
        if rc:
            raise ValueError("lso_teacher_logits_tail: bad arguments")
        return ex, fi

    def generate_full(self, prompt, max_new):
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(max_new, dtype=np.int32)
        mg, ma = np.zeros(max_new), np.zeros(max_new)
        n = C.c_int32()
        rc = lib().lso_generate_full(self._h, _ip(prompt), prompt.size, max_new, _ip(out),
                                     C.byref(n), _dp(mg), _dp(ma))
        if rc:
            raise ValueError("lso_generate_full: bad arguments")
        return out[:n.value], mg[:n.value], ma[:n.value]

    def generate_early(self, prompt, exit_layer, max_new):
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(max_new, dtype=np.int32)
        n = C.c_int32()
        rc = lib().lso_generate_early(self._h, _ip(prompt), prompt.size, exit_layer, max_new,
                                      _ip(out), C.byref(n))
        if rc:
            raise ValueError("lso_generate_early: bad arguments")
        return out[:n.value]

    def generate_adaptive(self, prompt, exit_layer, max_draft, min_margin, max_new):
        """Adaptive draft length: -> ids, accepted_per_step, drafted_per_step, and per step the
        smallest |exit-logit margin - min_margin| among the stop decisions it took."""
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(max_new, dtype=np.int32)
        acc = np.zeros(max_new, dtype=np.int32)
        dr = np.zeros(max_new, dtype=np.int32)
        gap = np.zeros(max_new, dtype=np.float64)
        n, s = C.c_int32(), C.c_int32()
        rc = lib().lso_generate_adaptive(self._h, _ip(prompt), prompt.size, exit_layer, max_draft,
                                         float(min_margin), max_new, _ip(out), C.byref(n), _ip(acc), _ip(dr),
                                         C.byref(s), gap.ctypes.data_as(C.POINTER(C.c_double)))
        if rc:
            raise ValueError("lso_generate_adaptive: bad arguments")
        return out[:n.value], acc[:s.value], dr[:s.value], gap[:s.value]

    def generate_spec(self, prompt, exit_layer, num_draft, max_new):
        """-> ids, accepted_per_step, cache_len after every step"""
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(max_new, dtype=np.int32)
        acc = np.zeros(max_new, dtype=np.int32)
        tr = np.zeros(max_new, dtype=np.int32)
        n, s = C.c_int32(), C.c_int32()
        rc = lib().lso_generate_spec(self._h, _ip(prompt), prompt.size, exit_layer, num_draft,
                                     max_new, _ip(out), C.byref(n), _ip(acc), C.byref(s), _ip(tr))
        if rc:
            raise ValueError("lso_generate_spec: bad arguments")
        return out[:n.value], acc[:s.value], tr[:s.value]
