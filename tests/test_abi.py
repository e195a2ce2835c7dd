"""The C-ABI library builds, loads and exports every symbol that include/ls.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import re
from pathlib import Path

from paper_2404_16710_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


def declared_functions():
    text = (ROOT / "include" / "ls.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ls_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = build.build()
    lib = ctypes.CDLL(str(lib_path))
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in ls.h but not exported"


def test_binding_covers_every_declared_symbol():
    assert sorted(binding.EXPORTS) == declared_functions()
    for n in binding.EXPORTS:
        if n not in ("ls_strerror", "ls_last_cuda_error"):
            assert callable(getattr(binding, n)), n


def test_host_only_calls_work_without_a_gpu():
    L = binding.lib()
    assert L.ls_strerror(0) == b"ok"
    assert b"capacity" in L.ls_strerror(binding.LS_ERR_CAPACITY)
    from paper_2404_16710_b200 import synth
    cfg = binding.make_config(synth.TINY, max_seq=128)
    n = binding.ls_workspace_bytes(cfg)
    kv = 2 * synth.TINY.n_layers * 128 * synth.TINY.kv_bytes_per_token_layer // 2
    assert n > kv and n % 256 == 0
    cfg.head_dim = 48  # not a shape the kernels cover
    assert binding.ls_workspace_bytes(cfg) == 0
    assert binding.ls_op_lm_head_scratch_bytes(32000) == 8 * 16 * 2000


def test_prompt_pass_ops_check_their_arguments_before_any_launch():
    """Argument errors of the prompt-pass entry points come back as codes, on the host (no GPU touched):
    this also pins the argument lists the binding declares for them."""
    L = binding.lib()
    bad = binding.LS_ERR_INVALID_ARG
    # q, R, pos0, Hq, Hkv, hd, page_size, page_table, max_seq, k_pages, v_pages, out, status, stream
    assert L.ls_op_prefill_attention(None, 0, 0, 8, 2, 128, 64, None, 4096, None, None, None, None, None) == bad
    assert L.ls_op_prefill_attention(None, 128, 0, 8, 3, 128, 64, None, 4096, None, None, None, None, None) == bad
    assert L.ls_op_prefill_attention(None, 128, 0, 8, 2, 96, 64, None, 4096, None, None, None, None, None) == bad
    assert L.ls_op_prefill_attention(None, 128, 0, 8, 2, 128, 48, None, 4096, None, None, None, None, None) == bad
    assert L.ls_op_prefill_attention(None, 128, 4000, 8, 2, 128, 64, None, 4096, None, None, None, None,
                                     None) == binding.LS_ERR_CAPACITY
    assert L.ls_op_prefill_attention(None, 128, 0, 8, 2, 128, 64, None, 4096, None, None, None, None, None) == bad  # null table
