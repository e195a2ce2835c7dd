"""The allocation-free LM-head + argmax entry point against the ordinary one.

Some callers of this library cannot allocate device memory and so cannot hand
ls_op_lm_head_argmax the scratch buffer it wants: code that runs while a stream is
being captured, plug-ins that are given a stream but no allocator, hosts with a closed,
pre-sized memory pool.  ls_op_lm_head_argmax_static keeps its scratch inside the library
instead.  Here it is called twice in a row (the second call finds the first call's
leftovers in the shared buffer) and must return exactly the token ids of the ordinary
entry point, which are integers and therefore compared bit for bit.

This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import pytest
import torch

from paper_2404_16710_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(seed, M, V, K):
    g = torch.Generator(device="cuda").manual_seed(seed)
    w = (torch.randn((V, K), generator=g, device="cuda") * 0.05).bfloat16()
    h = torch.randn((M, K), generator=g, device="cuda").bfloat16()
    return w, h


@pytest.mark.parametrize("path", [B.LS_LINEAR_FMA, B.LS_LINEAR_MMA])
def test_static_scratch_entry_point_matches_the_ordinary_one_twice_in_a_row(path):
    # first a wide vocabulary, then a narrower one with other data: stale candidates of the
    # first call sit beyond (and inside) the part of the buffer the second call uses
    for seed, M, V, K in ((1, 7, 32000, 512), (2, 16, 1000, 520)):
        w, h = _case(seed, M, V, K)
        scratch = torch.empty(B.ls_op_lm_head_scratch_bytes(V), dtype=torch.uint8, device="cuda")
        want = torch.full((M,), -1, dtype=torch.int32, device="cuda")
        got = torch.full((M,), -2, dtype=torch.int32, device="cuda")
        B.ls_op_lm_head_argmax(path, w, h, scratch, want, None)
        B.ls_op_lm_head_argmax_static(path, w, h, got)
        torch.cuda.synchronize()
        assert torch.equal(got, want), (seed, got.tolist(), want.tolist())
        assert int(want.min()) >= 0 and int(want.max()) < V


def test_static_scratch_entry_point_leaves_device_memory_as_it_is():
    """After a first call of the same configuration (which loads the kernel and looks the
    buffer's address up), a call changes neither the free device memory nor what torch has
    reserved: the entry point and everything under it allocate nothing."""
    w, h = _case(3, 5, 4096, 256)
    tok = torch.empty((5,), dtype=torch.int32, device="cuda")
    B.ls_op_lm_head_argmax_static(B.LS_LINEAR_MMA, w, h, tok)
    torch.cuda.synchronize()
    free0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
    B.ls_op_lm_head_argmax_static(B.LS_LINEAR_MMA, w, h, tok)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_reserved() == reserved0


def test_static_scratch_entry_point_refuses_a_vocabulary_beyond_its_buffer():
    V = B.LS_OP_LM_HEAD_STATIC_MAX_VOCAB + 16
    w = torch.zeros((V, 8), dtype=torch.bfloat16, device="cuda")
    h = torch.zeros((1, 8), dtype=torch.bfloat16, device="cuda")
    tok = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(B.LsError) as e:
        B.ls_op_lm_head_argmax_static(B.LS_LINEAR_MMA, w, h, tok)
    assert e.value.status == B.LS_ERR_CAPACITY
    torch.cuda.synchronize()
    assert int(tok[0]) == -7  # nothing ran
