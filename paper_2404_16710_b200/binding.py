"""Thin ctypes binding of the C ABI in ``include/ls.h`` -- argument marshalling only.

Every function has the name of the C entry point it calls.  Device operands are torch
CUDA tensors (only their ``data_ptr()`` crosses the boundary), host operands are numpy
arrays.  PyTorch is used for device memory and streams, nothing else: every step of the
path runs in the library's own kernels.  There is no fallback: if ``libls_b200.so`` is
missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import numpy as np

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libls_b200.so"

LS_OK = 0
LS_ERR_INVALID_ARG, LS_ERR_CAPACITY, LS_ERR_CUDA, LS_ERR_DEVICE_STATUS, LS_ERR_UNSUPPORTED = -1, -2, -3, -4, -5
LS_MAX_ROWS = 16
LS_LINEAR_AUTO, LS_LINEAR_FMA, LS_LINEAR_MMA = 0, 1, 2

EXPORTS = (
    "ls_strerror", "ls_last_cuda_error", "ls_workspace_bytes", "ls_model_create", "ls_model_destroy",
    "ls_set_page_table", "ls_generate", "ls_generate_adaptive", "ls_generate_full", "ls_generate_early", "ls_prefill",
    "ls_decode", "ls_decode_flags", "ls_decode_adaptive", "ls_read_output", "ls_read_drafted",
    "ls_generate_batch", "ls_prefill_batch", "ls_decode_batch", "ls_read_output_seq", "ls_debug_logits", "ls_debug_next_logits", "ls_get_stats", "ls_op_embed", "ls_op_rmsnorm",
    "ls_op_linear", "ls_op_gate_up_swiglu", "ls_op_lm_head_scratch_bytes", "ls_op_lm_head_argmax",
    "ls_op_lm_head_argmax_static", "ls_op_rope_append", "ls_op_qkv_rope_append", "ls_op_attention", "ls_op_accept",
    "ls_op_gemm", "ls_op_prefill_attention", "ls_op_chain",
)


class LsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ls_strerror(status).decode()
        if status == LS_ERR_CUDA:
            msg += f" [cudaError {lib().ls_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


class ls_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("vocab", C.c_int32), ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("max_seq", C.c_int32), ("page_size", C.c_int32), ("max_draft", C.c_int32),
                ("eos_id", C.c_int32), ("linear_path", C.c_int32)]


_VPP = C.POINTER(C.c_void_p)


class ls_weights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, _VPP) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class ls_stats(C.Structure):
    _fields_ = [("prefill_ms", C.c_double), ("decode_ms", C.c_double), ("weight_bytes", C.c_int64),
                ("kv_bytes", C.c_int64), ("kernel_launches", C.c_int64), ("n_generated", C.c_int32),
                ("n_steps", C.c_int32), ("n_accepted", C.c_int32), ("host_syncs", C.c_int32)]


_lib = None


def lib():
    """Load the CUDA library (built in-tree by ``paper_2404_16710_b200.build``)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2404_16710_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(str(LIB_PATH))
        i32, vp, ip, fp = C.c_int32, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float)
        sig = {
            "ls_strerror": (C.c_char_p, [C.c_int]),
            "ls_last_cuda_error": (C.c_int, []),
            "ls_workspace_bytes": (C.c_size_t, [C.POINTER(ls_config)]),
            "ls_model_create": (C.c_int, [C.POINTER(ls_config), C.POINTER(ls_weights), vp, C.c_size_t, vp,
                                          C.POINTER(vp)]),
            "ls_model_destroy": (C.c_int, [vp]),
            "ls_set_page_table": (C.c_int, [vp, ip, i32]),
            "ls_generate": (C.c_int, [vp, ip, i32, i32, i32, i32, ip, ip, ip, ip]),
            "ls_generate_full": (C.c_int, [vp, ip, i32, i32, ip, ip]),
            "ls_generate_early": (C.c_int, [vp, ip, i32, i32, i32, ip, ip]),
            "ls_prefill": (C.c_int, [vp, ip, i32, i32]),
            "ls_decode": (C.c_int, [vp, i32, i32, i32]),
            "ls_decode_flags": (C.c_int, [vp, i32, i32, i32, i32]),
            "ls_read_output": (C.c_int, [vp, ip, ip, ip, ip]),
            "ls_generate_batch": (C.c_int, [vp, i32, ip, ip, i32, i32, i32, ip, ip, ip, ip]),
            "ls_prefill_batch": (C.c_int, [vp, i32, ip, ip]),
            "ls_decode_batch": (C.c_int, [vp, i32, i32, i32]),
            "ls_read_output_seq": (C.c_int, [vp, i32, ip, ip, ip, ip]),
            "ls_generate_adaptive": (C.c_int, [vp, ip, i32, i32, i32, C.c_float, i32, ip, ip, ip, ip, ip]),
            "ls_decode_adaptive": (C.c_int, [vp, i32, i32, C.c_float, i32]),
            "ls_read_drafted": (C.c_int, [vp, ip, ip]),
            "ls_debug_logits": (C.c_int, [vp, ip, i32, i32, fp, fp]),
            "ls_debug_next_logits": (C.c_int, [vp, fp]),
            "ls_get_stats": (C.c_int, [vp, C.POINTER(ls_stats)]),
            "ls_op_chain": (C.c_int, [i32]),
            "ls_op_embed": (C.c_int, [vp, vp, i32, i32, i32, vp, vp]),
            "ls_op_rmsnorm": (C.c_int, [vp, vp, i32, i32, C.c_float, vp, vp]),
            "ls_op_linear": (C.c_int, [i32, vp, vp, i32, i32, i32, vp, i32, vp]),
            "ls_op_gate_up_swiglu": (C.c_int, [i32, vp, vp, vp, i32, i32, i32, vp, vp]),
            "ls_op_lm_head_scratch_bytes": (C.c_size_t, [i32]),
            "ls_op_lm_head_argmax": (C.c_int, [i32, vp, vp, i32, i32, i32, vp, vp, vp, vp]),
            "ls_op_lm_head_argmax_static": (C.c_int, [i32, vp, vp, i32, i32, i32, vp, vp]),
            "ls_op_rope_append": (C.c_int, [vp, i32, i32, i32, i32, i32, C.c_float, i32, vp, i32, vp, vp, vp, vp]),
            "ls_op_qkv_rope_append": (C.c_int, [i32, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, C.c_float, i32, vp, i32,
                                                vp, vp, vp, vp]),
            "ls_op_attention": (C.c_int, [vp, i32, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp, vp]),
            "ls_op_accept": (C.c_int, [vp, vp, i32, vp, vp, vp, vp]),
            "ls_op_gemm": (C.c_int, [vp, vp, i32, i32, i32, vp, i32, i32, vp, vp]),
            "ls_op_prefill_attention": (C.c_int, [vp, i32, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp, vp, vp]),
        }
        for name, (res, args) in sig.items():
            f = getattr(L, name)
            f.restype, f.argtypes = res, args
        _lib = L
    return _lib


def _ck(rc, where):
    if rc != LS_OK:
        raise LsError(rc, where)


def _dev(t):
    """device pointer of a torch CUDA tensor (None -> NULL)"""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


# ------------------------------------------------------------------ model-level entry points
def make_config(shape, max_seq, page_size=64, max_draft=8, eos_id=-1, linear_path=LS_LINEAR_AUTO) -> ls_config:
    """shape: any object with the decoder-shape attributes (e.g. synth.Shape)."""
    return ls_config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim,
                     shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta, max_seq, page_size,
                     max_draft, eos_id, linear_path)


def ls_workspace_bytes(cfg: ls_config) -> int:
    return lib().ls_workspace_bytes(C.byref(cfg))


def ls_model_create(cfg: ls_config, weights: dict, workspace, stream=None):
    """weights: dict of torch bf16 CUDA tensors (per-layer entries are lists).  Returns the
    opaque handle; the caller keeps ``weights`` and ``workspace`` alive."""
    w = ls_weights()
    keep = []
    for k in ("tok_embed", "final_norm", "lm_head"):
        setattr(w, k, weights[k].data_ptr())
    for k in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
        arr = (C.c_void_p * cfg.n_layers)(*[t.data_ptr() for t in weights[k]])
        keep.append(arr)
        setattr(w, k, C.cast(arr, _VPP))
    h = C.c_void_p()
    st = C.c_void_p(stream) if stream else None  # None: the model makes a stream of its own
    _ck(lib().ls_model_create(C.byref(cfg), C.byref(w), _dev(workspace), workspace.numel() * workspace.element_size(),
                              st, C.byref(h)), "ls_model_create")
    return h


def ls_model_destroy(h):
    _ck(lib().ls_model_destroy(h), "ls_model_destroy")


def ls_set_page_table(h, table):
    a, p = _i32(table)
    _ck(lib().ls_set_page_table(h, p, a.size), "ls_set_page_table")


def ls_generate(h, prompt, exit_layer, num_draft, max_new):
    """-> (ids, accepted_per_step) as numpy int32 arrays"""
    a, p = _i32(prompt)
    out, acc = np.zeros(max_new, np.int32), np.zeros(max_new, np.int32)
    n, s = C.c_int32(), C.c_int32()
    _ck(lib().ls_generate(h, p, a.size, exit_layer, num_draft, max_new,
                          out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(n),
                          acc.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(s)), "ls_generate")
    return out[:n.value], acc[:s.value]


def ls_generate_adaptive(h, prompt, exit_layer, max_draft, min_margin, max_new):
    """-> (ids, accepted_per_step, drafted_per_step) as numpy int32 arrays"""
    a, p = _i32(prompt)
    out, acc, dr = np.zeros(max_new, np.int32), np.zeros(max_new, np.int32), np.zeros(max_new, np.int32)
    n, s = C.c_int32(), C.c_int32()
    ip = C.POINTER(C.c_int32)
    _ck(lib().ls_generate_adaptive(h, p, a.size, exit_layer, max_draft, float(min_margin), max_new,
                                   out.ctypes.data_as(ip), C.byref(n), acc.ctypes.data_as(ip),
                                   dr.ctypes.data_as(ip), C.byref(s)), "ls_generate_adaptive")
    return out[:n.value], acc[:s.value], dr[:s.value]


def ls_generate_full(h, prompt, max_new):
    a, p = _i32(prompt)
    out = np.zeros(max_new, np.int32)
    n = C.c_int32()
    _ck(lib().ls_generate_full(h, p, a.size, max_new, out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(n)),
        "ls_generate_full")
    return out[:n.value]


def ls_generate_early(h, prompt, exit_layer, max_new):
    a, p = _i32(prompt)
    out = np.zeros(max_new, np.int32)
    n = C.c_int32()
    _ck(lib().ls_generate_early(h, p, a.size, exit_layer, max_new, out.ctypes.data_as(C.POINTER(C.c_int32)),
                                C.byref(n)), "ls_generate_early")
    return out[:n.value]


def ls_prefill(h, prompt, layers=0):
    a, p = _i32(prompt)
    _ck(lib().ls_prefill(h, p, a.size, layers), "ls_prefill")


def ls_decode(h, exit_layer, num_draft, max_new):
    _ck(lib().ls_decode(h, exit_layer, num_draft, max_new), "ls_decode")


LS_DECODE_NO_EXIT_CACHE = 1


def ls_decode_flags(h, exit_layer, num_draft, max_new, flags):
    _ck(lib().ls_decode_flags(h, exit_layer, num_draft, max_new, flags), "ls_decode_flags")


def ls_decode_adaptive(h, exit_layer, max_draft, min_margin, max_new):
    _ck(lib().ls_decode_adaptive(h, exit_layer, max_draft, float(min_margin), max_new), "ls_decode_adaptive")


def ls_read_drafted(h, max_new):
    dr = np.zeros(max_new, np.int32)
    s = C.c_int32()
    _ck(lib().ls_read_drafted(h, dr.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(s)), "ls_read_drafted")
    return dr[:s.value]


def ls_read_output(h, max_new):
    out, acc = np.zeros(max_new, np.int32), np.zeros(max_new, np.int32)
    n, s = C.c_int32(), C.c_int32()
    _ck(lib().ls_read_output(h, out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(n),
                             acc.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(s)), "ls_read_output")
    return out[:n.value], acc[:s.value]


def _cat_prompts(prompts):
    lens = np.asarray([len(p) for p in prompts], dtype=np.int32)
    flat = np.ascontiguousarray(np.concatenate([np.asarray(p, dtype=np.int32) for p in prompts]))
    return flat, lens


def ls_prefill_batch(h, prompts):
    flat, lens = _cat_prompts(prompts)
    ipt = C.POINTER(C.c_int32)
    _ck(lib().ls_prefill_batch(h, len(prompts), flat.ctypes.data_as(ipt), lens.ctypes.data_as(ipt)), "ls_prefill_batch")


def ls_decode_batch(h, exit_layer, num_draft, max_new):
    _ck(lib().ls_decode_batch(h, exit_layer, num_draft, max_new), "ls_decode_batch")


def ls_read_output_seq(h, seq, max_new):
    out, acc = np.zeros(max_new, np.int32), np.zeros(max_new, np.int32)
    n, s = C.c_int32(), C.c_int32()
    ipt = C.POINTER(C.c_int32)
    _ck(lib().ls_read_output_seq(h, seq, out.ctypes.data_as(ipt), C.byref(n), acc.ctypes.data_as(ipt), C.byref(s)),
        "ls_read_output_seq")
    return out[:n.value], acc[:s.value]


def ls_generate_batch(h, prompts, exit_layer, num_draft, max_new):
    """-> [(ids, accepted_per_step)] per sequence"""
    flat, lens = _cat_prompts(prompts)
    B = len(prompts)
    out, acc = np.zeros((B, max_new), np.int32), np.zeros((B, max_new), np.int32)
    n, st = np.zeros(B, np.int32), np.zeros(B, np.int32)
    ipt = C.POINTER(C.c_int32)
    _ck(lib().ls_generate_batch(h, B, flat.ctypes.data_as(ipt), lens.ctypes.data_as(ipt), exit_layer, num_draft, max_new,
                                out.ctypes.data_as(ipt), n.ctypes.data_as(ipt), acc.ctypes.data_as(ipt),
                                st.ctypes.data_as(ipt)), "ls_generate_batch")
    return [(out[b, :n[b]].copy(), acc[b, :st[b]].copy()) for b in range(B)]


def ls_debug_next_logits(h, vocab):
    """after ls_prefill: final logits of the last prompt token on top of the prompt pass's cache"""
    out = np.empty(vocab, np.float32)
    _ck(lib().ls_debug_next_logits(h, out.ctypes.data_as(C.POINTER(C.c_float))), "ls_debug_next_logits")
    return out


def ls_debug_logits(h, ids, exit_layer, vocab, want_exit=True, want_final=True):
    a, p = _i32(ids)
    ex = np.empty((a.size, vocab), np.float32) if want_exit else None
    fi = np.empty((a.size, vocab), np.float32) if want_final else None
    fp = C.POINTER(C.c_float)
    _ck(lib().ls_debug_logits(h, p, a.size, exit_layer, ex.ctypes.data_as(fp) if want_exit else None,
                              fi.ctypes.data_as(fp) if want_final else None), "ls_debug_logits")
    return ex, fi


def ls_get_stats(h) -> ls_stats:
    s = ls_stats()
    _ck(lib().ls_get_stats(h, C.byref(s)), "ls_get_stats")
    return s


# ------------------------------------------------------------------ single operations (torch CUDA tensors)
def ls_op_embed(emb, tok, x):
    M, D = x.shape
    _ck(lib().ls_op_embed(_dev(emb), _dev(tok), M, D, emb.shape[0], _dev(x), _stream()), "ls_op_embed")


def ls_op_rmsnorm(x, gain, eps, out):
    M, D = x.shape
    _ck(lib().ls_op_rmsnorm(_dev(x), _dev(gain), M, D, eps, _dev(out), _stream()), "ls_op_rmsnorm")


def ls_op_chain(on):
    _ck(lib().ls_op_chain(int(bool(on))), "ls_op_chain")


def ls_op_linear(path, w, h, out, residual=False):
    (N, K), M = w.shape, h.shape[0]
    _ck(lib().ls_op_linear(path, _dev(w), _dev(h), M, N, K, _dev(out), int(residual), _stream()), "ls_op_linear")


def ls_op_gate_up_swiglu(path, w_gate, w_up, h, out):
    (F, K), M = w_gate.shape, h.shape[0]
    _ck(lib().ls_op_gate_up_swiglu(path, _dev(w_gate), _dev(w_up), _dev(h), M, F, K, _dev(out), _stream()),
        "ls_op_gate_up_swiglu")


def ls_op_lm_head_scratch_bytes(V):
    return lib().ls_op_lm_head_scratch_bytes(V)


def ls_op_lm_head_argmax(path, w, h, scratch, tok, logits=None):
    (V, K), M = w.shape, h.shape[0]
    _ck(lib().ls_op_lm_head_argmax(path, _dev(w), _dev(h), M, V, K, _dev(scratch), _dev(tok), _dev(logits),
                                   _stream()), "ls_op_lm_head_argmax")


LS_OP_LM_HEAD_STATIC_MAX_VOCAB = 131072


def ls_op_lm_head_argmax_static(path, w, h, tok):
    """LM head + argmax for callers that have no scratch buffer to give (they cannot
    allocate): the candidates go to a buffer inside the library.  Vocabulary at most
    LS_OP_LM_HEAD_STATIC_MAX_VOCAB; calls must not overlap on the GPU."""
    (V, K), M = w.shape, h.shape[0]
    _ck(lib().ls_op_lm_head_argmax_static(path, _dev(w), _dev(h), M, V, K, _dev(tok), _stream()),
        "ls_op_lm_head_argmax_static")


def ls_op_rope_append(qkv, pos0, Hq, Hkv, hd, theta, page_size, page_table, max_seq, q_out, k_pages, v_pages):
    _ck(lib().ls_op_rope_append(_dev(qkv), qkv.shape[0], pos0, Hq, Hkv, hd, theta, page_size, _dev(page_table),
                                max_seq, _dev(q_out), _dev(k_pages), _dev(v_pages), _stream()), "ls_op_rope_append")


def ls_op_qkv_rope_append(path, wq, wk, wv, h, pos0, Hq, Hkv, hd, theta, page_size, page_table, max_seq, q_out,
                          k_pages, v_pages):
    M, K = h.shape
    _ck(lib().ls_op_qkv_rope_append(path, _dev(wq), _dev(wk), _dev(wv), _dev(h), M, K, pos0, Hq, Hkv, hd, theta,
                                    page_size, _dev(page_table), max_seq, _dev(q_out), _dev(k_pages), _dev(v_pages),
                                    _stream()), "ls_op_qkv_rope_append")


def ls_op_attention(q, pos0, Hq, Hkv, hd, page_size, page_table, max_seq, k_pages, v_pages, out):
    _ck(lib().ls_op_attention(_dev(q), q.shape[0], pos0, Hq, Hkv, hd, page_size, _dev(page_table), max_seq,
                              _dev(k_pages), _dev(v_pages), _dev(out), _stream()), "ls_op_attention")


def ls_op_gemm(a, b, c, accumulate=False, status=None):
    """c[M, N] (+)= a[M, K] @ b[N, K].T  (bf16 inputs, fp32 c, tcgen05 tensor cores)"""
    (M, K), N = a.shape, b.shape[0]
    _ck(lib().ls_op_gemm(_dev(a), _dev(b), M, N, K, _dev(c), c.stride(0), int(accumulate), _dev(status), _stream()),
        "ls_op_gemm")


def ls_op_prefill_attention(q, pos0, Hq, Hkv, hd, page_size, page_table, max_seq, k_pages, v_pages, out, status=None):
    _ck(lib().ls_op_prefill_attention(_dev(q), q.shape[0], pos0, Hq, Hkv, hd, page_size, _dev(page_table), max_seq,
                                      _dev(k_pages), _dev(v_pages), _dev(out), _dev(status), _stream()),
        "ls_op_prefill_attention")


def ls_op_accept(draft, verified, d, state, out_ids, accepted):
    _ck(lib().ls_op_accept(_dev(draft), _dev(verified), d, _dev(state), _dev(out_ids), _dev(accepted), _stream()),
        "ls_op_accept")


# ------------------------------------------------------------------ convenience: own the device memory of one model
class Model:
    """Allocates the workspace with torch, creates the handle, keeps everything alive."""

    def __init__(self, shape, weights: dict, max_seq: int, page_size: int = 64, max_draft: int = 8,
                 eos_id: int = -1, linear_path: int = LS_LINEAR_AUTO):
        import torch
        self.shape = shape
        self.cfg = make_config(shape, max_seq, page_size, max_draft, eos_id, linear_path)
        nbytes = ls_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise LsError(LS_ERR_INVALID_ARG, "ls_workspace_bytes")
        self.weights = weights
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.h = ls_model_create(self.cfg, weights, self.workspace)

    def close(self):
        if getattr(self, "h", None):
            ls_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def generate(self, prompt, exit_layer, num_draft, max_new):
        return ls_generate(self.h, prompt, exit_layer, num_draft, max_new)

    def generate_adaptive(self, prompt, exit_layer, max_draft, min_margin, max_new):
        return ls_generate_adaptive(self.h, prompt, exit_layer, max_draft, min_margin, max_new)

    def generate_full(self, prompt, max_new):
        return ls_generate_full(self.h, prompt, max_new)

    def generate_early(self, prompt, exit_layer, max_new):
        return ls_generate_early(self.h, prompt, exit_layer, max_new)

    def generate_batch(self, prompts, exit_layer, num_draft, max_new):
        return ls_generate_batch(self.h, prompts, exit_layer, num_draft, max_new)

    def debug_logits(self, ids, exit_layer, want_exit=True, want_final=True):
        return ls_debug_logits(self.h, ids, exit_layer, self.shape.vocab, want_exit, want_final)

    def stats(self):
        return ls_get_stats(self.h)
