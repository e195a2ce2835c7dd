"""Parity of every kernel family against the oracle's elementary operation, through the C ABI.

Sizes span several tiles and a ragged tail (rows not a multiple of 16, K not a multiple
of 32, M from 1 to 16), plus the full Llama-2-7B projection shapes checked on sampled
output rows.  Integer results (token ids, accept bookkeeping) must be bit-exact; floating
point results carry the tolerance their arithmetic implies: fp32 accumulation of exact
bf16 products against the oracle's fp64 (1e-5 relative to the row's magnitude), one bf16
rounding (2^-8 relative) where the kernel's output is bf16.
"""
import math

import numpy as np
import pytest
import torch

from oracle import ls_oracle as O
from paper_2404_16710_b200 import binding as B
from tests.helpers import bf16_cuda, bits, vals

pytestmark = pytest.mark.gpu
PATHS = [B.LS_LINEAR_FMA, B.LS_LINEAR_MMA]
BF16_REL = 2.0 ** -8


def rnd(shape, seed, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(shape, generator=g, device="cuda") * scale)


def assert_bf16_close(got, ref, what=""):
    tol = BF16_REL * np.abs(ref) + 1e-6 * np.abs(ref).max()
    bad = np.abs(got - ref) > tol
    assert not bad.any(), f"{what}: {bad.sum()} elements off, worst {np.abs(got - ref).max():.4g}"


# ------------------------------------------------------------------ embedding, RMSNorm
def test_embed_is_a_row_lookup():
    emb = rnd((50, 64), 1).bfloat16()
    tok = torch.tensor([3, 49, 0, 3, 17], dtype=torch.int32, device="cuda")
    x = torch.empty((5, 64), dtype=torch.float32, device="cuda")
    B.ls_op_embed(emb, tok, x)
    torch.cuda.synchronize()
    assert torch.equal(x, emb[tok.long()].float())


@pytest.mark.parametrize("M,D", [(1, 64), (3, 256), (16, 4096), (7, 5120), (2, 1000)])
def test_rmsnorm(M, D):
    x = rnd((M, D), 2, 3.0)
    g = (1 + 0.1 * rnd((D,), 3)).bfloat16()
    out = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
    B.ls_op_rmsnorm(x, g, 1e-5, out)
    torch.cuda.synchronize()
    xs, gb = x.cpu().numpy().astype(np.float64), bits(g)
    for m in range(M):
        assert_bf16_close(vals(out[m]), O.rmsnorm(xs[m], gb, 1e-5), f"row {m}")


# ------------------------------------------------------------------ linear families
def linear_case(path, M, N, K, residual, seed):
    w = rnd((N, K), seed, 0.05).bfloat16()
    h = rnd((M, K), seed + 1).bfloat16()
    out = rnd((M, N), seed + 2) if residual else torch.empty((M, N), dtype=torch.float32, device="cuda")
    base = out.clone()
    B.ls_op_linear(path, w, h, out, residual)
    torch.cuda.synchronize()
    return w, h, base, out


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,N,K", [(1, 16, 32), (1, 200, 88), (3, 100, 256), (4, 256, 688), (7, 333, 1000),
                                   (8, 64, 4096), (9, 48, 72), (16, 130, 520)])
@pytest.mark.parametrize("residual", [False, True])
def test_linear_small_shapes(path, M, N, K, residual):
    w, h, base, out = linear_case(path, M, N, K, residual, 10 + M)
    wb, hv = bits(w), vals(h)
    got = out.cpu().numpy().astype(np.float64)
    for m in range(M):
        ref = O.linear(wb, hv[m]) + (base[m].cpu().numpy() if residual else 0.0)
        np.testing.assert_allclose(got[m], ref, rtol=0, atol=1e-5 * np.abs(ref).max() + 1e-6)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("N,K", [(12288, 4096), (4096, 11008), (4096, 4096)])
def test_linear_llama7b_shapes_sampled_rows(path, N, K):
    M = 7
    w, h, _, out = linear_case(path, M, N, K, False, 77)
    rows = np.unique(np.concatenate([[0, 15, 16, N - 17, N - 1],
                                     np.random.default_rng(0).integers(0, N, 40)]))
    wb, hv = bits(w[torch.from_numpy(rows).cuda()]), vals(h)
    got = out.cpu().numpy().astype(np.float64)[:, rows]
    for m in range(M):
        ref = O.linear(wb, hv[m])
        np.testing.assert_allclose(got[m], ref, rtol=0, atol=1e-5 * np.abs(ref).max())


@pytest.mark.parametrize("path", PATHS)
def test_linear_rows_do_not_depend_on_pass_size(path):
    """Row 0 of an M-row pass is bit-identical for every M (the verification pass must
    reproduce single-token decoding exactly)."""
    N, K = 304, 1384
    w = rnd((N, K), 5, 0.05).bfloat16()
    h = rnd((16, K), 6).bfloat16()
    outs = {}
    for M in (1, 2, 4, 5, 8, 9, 16):
        out = torch.empty((M, N), dtype=torch.float32, device="cuda")
        B.ls_op_linear(path, w, h[:M].contiguous(), out)
        outs[M] = out
    torch.cuda.synchronize()
    for M, out in outs.items():
        assert torch.equal(out[0], outs[1][0]), f"M={M}"
        assert torch.equal(out[M - 1], outs[16][M - 1]), f"M={M}"
    # and a row's value does not depend on which slot of the pass it occupies
    hh = h[:9].flip(0).contiguous()
    out = torch.empty((9, N), dtype=torch.float32, device="cuda")
    B.ls_op_linear(path, w, hh, out)
    torch.cuda.synchronize()
    assert torch.equal(out.flip(0), outs[9])


def test_chained_operations_give_the_same_results():
    """ls_op_chain(1): consecutive operations overlap as they do inside the decode loop (a kernel
    moves in while its predecessor finishes and waits before it reads the predecessor's output).
    A dependent sequence -- three residual updates of one buffer, then gate-up on another --
    gives bit-identical results either way."""
    path = B.LS_LINEAR_MMA
    N = K = 1024
    ws = [rnd((N, K), 40 + i, 0.05).bfloat16() for i in range(3)]
    wg, wu = rnd((704, K), 50, 0.05).bfloat16(), rnd((704, K), 51, 0.05).bfloat16()
    h = rnd((5, K), 44).bfloat16()
    outs = []
    for on in (False, True, False):
        B.ls_op_chain(on)
        try:
            x = torch.zeros((5, N), dtype=torch.float32, device="cuda")
            act = torch.empty((5, 704), dtype=torch.bfloat16, device="cuda")
            for w in ws:
                B.ls_op_linear(path, w, h, x, True)
            B.ls_op_gate_up_swiglu(path, wg, wu, h, act)
            torch.cuda.synchronize()
        finally:
            B.ls_op_chain(False)
        outs.append((x, act))
    for x, act in outs[1:]:
        assert torch.equal(x, outs[0][0]) and torch.equal(act, outs[0][1])


@pytest.mark.parametrize("residual", [False, True])
@pytest.mark.parametrize("N,K", [(4096, 4096), (5120, 1024), (4100, 520)])
def test_wide_matrices_cut_per_sm_give_the_same_rows(N, K, residual):
    """From 9 rows on the wide matrices (o-proj and down-proj shapes) are cut into one share of
    rows per SM instead of one 16-row tile per CTA; shares are ragged (4096 / 148 rows). Every
    output row is bit-identical to what the single-row pass gives, at every pass size on both
    sides of the switch, with and without the residual add; sampled rows against the oracle."""
    path = B.LS_LINEAR_MMA
    w = rnd((N, K), 31, 0.05).bfloat16()
    h = rnd((16, K), 32).bfloat16()
    x0 = rnd((16, N), 33)
    single = torch.empty((16, N), dtype=torch.float32, device="cuda")
    for m in range(16):
        o = x0[m:m + 1].clone() if residual else torch.empty((1, N), dtype=torch.float32, device="cuda")
        B.ls_op_linear(path, w, h[m:m + 1].contiguous(), o, residual)
        single[m] = o[0]
    for M in (8, 9, 11, 16):
        out = x0[:M].clone() if residual else torch.empty((M, N), dtype=torch.float32, device="cuda")
        B.ls_op_linear(path, w, h[:M].contiguous(), out, residual)
        torch.cuda.synchronize()
        assert torch.equal(out, single[:M]), f"M={M}"
    rows = np.unique(np.concatenate([[0, 26, 27, 28, 55, N - 29, N - 1], np.random.default_rng(3).integers(0, N, 24)]))
    wb, hv = bits(w[torch.from_numpy(rows).cuda()]), vals(h)
    got = single.cpu().numpy().astype(np.float64)[:, rows]
    base = x0.cpu().numpy().astype(np.float64)[:, rows] if residual else 0.0
    for m in (0, 9, 15):
        ref = O.linear(wb, hv[m]) + (base[m] if residual else 0.0)
        np.testing.assert_allclose(got[m], ref, rtol=0, atol=2e-5 * np.abs(ref).max())


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,F,K", [(1, 8, 32), (3, 88, 96), (7, 688, 256), (16, 100, 520), (5, 11008, 4096)])
def test_gate_up_swiglu(path, M, F, K):
    wg, wu = rnd((F, K), 20, 0.05).bfloat16(), rnd((F, K), 21, 0.05).bfloat16()
    h = rnd((M, K), 22).bfloat16()
    out = torch.empty((M, F), dtype=torch.bfloat16, device="cuda")
    B.ls_op_gate_up_swiglu(path, wg, wu, h, out)
    torch.cuda.synchronize()
    cols = np.arange(F) if F <= 1000 else np.unique(np.concatenate(
        [[0, 7, 8, F - 9, F - 1], np.random.default_rng(1).integers(0, F, 48)]))
    idx = torch.from_numpy(cols).cuda()
    gb, ub, hv = bits(wg[idx]), bits(wu[idx]), vals(h)
    for m in range(M):
        g, u = O.linear(gb, hv[m]), O.linear(ub, hv[m])
        ref = np.array([O.silu(a) for a in g]) * u
        assert_bf16_close(vals(out[m])[cols], ref, f"row {m}")


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,V,K", [(1, 200, 96), (4, 1024, 256), (7, 32000, 4096), (16, 1000, 520)])
def test_lm_head_argmax(path, M, V, K):
    w = rnd((V, K), 30, 0.05).bfloat16()
    h = rnd((M, K), 31).bfloat16()
    scratch = torch.empty(B.ls_op_lm_head_scratch_bytes(V), dtype=torch.uint8, device="cuda")
    tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    logits = torch.empty((M, V), dtype=torch.float32, device="cuda")
    B.ls_op_lm_head_argmax(path, w, h, scratch, tok, logits)
    tok2 = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    B.ls_op_lm_head_argmax(path, w, h, scratch, tok2, None)
    torch.cuda.synchronize()
    assert torch.equal(tok, tok2)
    wb, hv = bits(w), vals(h)
    lg = logits.cpu().numpy().astype(np.float64)
    for m in range(M):
        ref = O.linear(wb, hv[m])
        np.testing.assert_allclose(lg[m], ref, rtol=0, atol=1e-5 * np.abs(ref).max())
        # the id is the argmax of the kernel's own fp32 logits (ties -> lowest index) ...
        assert int(tok[m]) == int(np.argmax(logits[m].cpu().numpy()))
        # ... and the oracle's id whenever the oracle's margin is beyond fp32 accumulation error
        i, margin, ma = O.argmax(ref)
        if margin > 2e-5 * ma:
            assert int(tok[m]) == i


@pytest.mark.parametrize("path", PATHS)
def test_lm_head_argmax_tie_goes_to_lowest_index(path):
    V, K = 96, 64
    w = torch.zeros((V, K), dtype=torch.bfloat16, device="cuda")
    w[[5, 37, 70], 0] = 2.0   # three equal maxima in different tiles
    w[11, 0] = 1.0
    h = torch.zeros((2, K), dtype=torch.bfloat16, device="cuda")
    h[0, 0], h[1, 0] = 1.0, -1.0  # row 1: all of {5,37,70,11} negative, the zeros tie at 0 -> index 0
    scratch = torch.empty(B.ls_op_lm_head_scratch_bytes(V), dtype=torch.uint8, device="cuda")
    tok = torch.empty((2,), dtype=torch.int32, device="cuda")
    B.ls_op_lm_head_argmax(path, w, h, scratch, tok, None)
    torch.cuda.synchronize()
    assert tok.tolist() == [5, 0]


# ------------------------------------------------------------------ RoPE + append, attention
def kv_setup(Hkv, hd, page_size, max_seq, shuffle):
    n_pages = -(-max_seq // page_size)
    table = np.arange(n_pages, dtype=np.int32)
    if shuffle:
        table = np.random.default_rng(3).permutation(n_pages).astype(np.int32)
    kp = torch.zeros((n_pages, Hkv, page_size, hd), dtype=torch.bfloat16, device="cuda")
    vp = torch.zeros_like(kp)
    return table, torch.from_numpy(table).cuda(), kp, vp


def gather_cache(pages, table, page_size, n):
    """[n, Hkv*hd] float64 rows of logical positions 0..n-1"""
    rows = []
    for p in range(n):
        phys = table[p // page_size]
        rows.append(vals(pages[phys, :, p % page_size, :]).reshape(-1))
    return np.stack(rows)


@pytest.mark.parametrize("Hq,Hkv,hd,theta", [(4, 2, 64, 1e4), (8, 8, 128, 1e4), (8, 2, 128, 5e5)])
@pytest.mark.parametrize("shuffle", [False, True])
def test_rope_append(Hq, Hkv, hd, theta, shuffle):
    M, pos0, page_size, max_seq = 5, 1021, 16, 1100
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, shuffle)
    qkv = rnd((M, (Hq + 2 * Hkv) * hd), 40)
    q_out = torch.empty((M, Hq * hd), dtype=torch.bfloat16, device="cuda")
    B.ls_op_rope_append(qkv, pos0, Hq, Hkv, hd, theta, page_size, table_d, max_seq, q_out, kp, vp)
    torch.cuda.synchronize()
    src = qkv.cpu().numpy().astype(np.float64)
    kc = gather_cache(kp, table, page_size, pos0 + M)
    vc = gather_cache(vp, table, page_size, pos0 + M)
    assert not kc[:pos0].any() and not vc[:pos0].any()  # nothing else was touched
    for m in range(M):
        p = pos0 + m
        for hh in range(Hq):
            ref = O.rope(src[m, hh * hd:(hh + 1) * hd], p, theta)
            # fp32 angle p * inv_freq carries ~p * 2^-24 radians of error on top of the bf16 rounding
            np.testing.assert_allclose(vals(q_out[m, hh * hd:(hh + 1) * hd]), ref, rtol=0,
                                       atol=BF16_REL * np.abs(ref).max() + 4e-4 * np.abs(ref).max())
        for hh in range(Hkv):
            o = (Hq + hh) * hd
            ref = O.rope(src[m, o:o + hd], p, theta)
            np.testing.assert_allclose(kc[p, hh * hd:(hh + 1) * hd], ref, rtol=0,
                                       atol=(BF16_REL + 4e-4) * np.abs(ref).max())
            o = (Hq + Hkv + hh) * hd
            ref = src[m, o:o + hd]
            assert_bf16_close(vc[p, hh * hd:(hh + 1) * hd], ref)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("Hq,Hkv,hd,K,M", [(4, 2, 64, 96, 5), (8, 8, 128, 256, 1), (8, 2, 128, 520, 9)])
def test_qkv_projection_fused_with_rope_and_append(path, Hq, Hkv, hd, K, M):
    """What the decode loop runs: q|k|v projection, rotary embedding and cache append in one kernel."""
    pos0, page_size, max_seq, theta = 77, 16, 160, 1e4
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, True)
    wq, wk, wv = (rnd((n, K), 70 + i, 0.05).bfloat16() for i, n in enumerate((Hq * hd, Hkv * hd, Hkv * hd)))
    h = rnd((M, K), 73).bfloat16()
    q_out = torch.empty((M, Hq * hd), dtype=torch.bfloat16, device="cuda")
    B.ls_op_qkv_rope_append(path, wq, wk, wv, h, pos0, Hq, Hkv, hd, theta, page_size, table_d, max_seq, q_out, kp, vp)
    torch.cuda.synchronize()
    kc = gather_cache(kp, table, page_size, pos0 + M)
    vc = gather_cache(vp, table, page_size, pos0 + M)
    assert not kc[:pos0].any() and not vc[:pos0].any()
    hv = vals(h)
    for m in range(M):
        p = pos0 + m
        qr, kr, vr = O.linear(bits(wq), hv[m]), O.linear(bits(wk), hv[m]), O.linear(bits(wv), hv[m])
        for hh in range(Hq):
            ref = O.rope(qr[hh * hd:(hh + 1) * hd], p, theta)
            np.testing.assert_allclose(vals(q_out[m, hh * hd:(hh + 1) * hd]), ref, rtol=0,
                                       atol=(BF16_REL + 1e-4) * np.abs(ref).max())
        for hh in range(Hkv):
            ref = O.rope(kr[hh * hd:(hh + 1) * hd], p, theta)
            np.testing.assert_allclose(kc[p, hh * hd:(hh + 1) * hd], ref, rtol=0,
                                       atol=(BF16_REL + 1e-4) * np.abs(ref).max())
            ref = vr[hh * hd:(hh + 1) * hd]
            np.testing.assert_allclose(vc[p, hh * hd:(hh + 1) * hd], ref, rtol=0,
                                       atol=(BF16_REL + 1e-5) * np.abs(ref).max())


def attention_tol(q, k, v, Hq, Hkv, hd, ref):
    """Elementwise bound on |kernel - oracle| for one query row.  The kernels feed the softmax
    weights to the tensor cores as bf16 (relative error <= 2^-9 each) while the normalising
    sum stays fp32, so output j moves by at most 2^-9 * sum_i a_i |v_ij| -- the attention
    output of |v| -- and the bf16 result then rounds once more (BF16_REL of the largest
    output covers that and the fp32 accumulation)."""
    spread = O.attention(q, k, np.abs(v), Hq, Hkv, hd)
    return BF16_REL * np.abs(ref).max() + 2.0 ** -9 * spread + 1e-5


@pytest.mark.parametrize("Hq,Hkv,hd", [(4, 2, 64), (4, 4, 128), (8, 2, 128)])
@pytest.mark.parametrize("M,pos0", [(1, 0), (1, 63), (1, 64), (4, 61), (7, 130), (16, 300), (3, 1000)])
def test_attention(Hq, Hkv, hd, M, pos0):
    page_size, max_seq = 32, 1100
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, True)
    n = pos0 + M
    # fill logical positions 0..n-1 (and garbage beyond, which causal masking must hide)
    kl = rnd((n + 8, Hkv, hd), 50).bfloat16()
    vl = rnd((n + 8, Hkv, hd), 51).bfloat16()
    for p in range(min(n + 8, max_seq)):
        kp[table[p // page_size], :, p % page_size, :] = kl[p]
        vp[table[p // page_size], :, p % page_size, :] = vl[p]
    q = rnd((M, Hq * hd), 52, 0.5).bfloat16()
    out = torch.empty((M, Hq * hd), dtype=torch.bfloat16, device="cuda")
    B.ls_op_attention(q, pos0, Hq, Hkv, hd, page_size, table_d, max_seq, kp, vp, out)
    torch.cuda.synchronize()
    kf, vf, qf = vals(kl).reshape(n + 8, -1), vals(vl).reshape(n + 8, -1), vals(q)
    for m in range(M):
        ref = O.attention(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd)
        assert (np.abs(vals(out[m]) - ref) <= attention_tol(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd, ref)).all()


def test_attention_rows_do_not_depend_on_pass_size():
    Hq, Hkv, hd, page_size, max_seq, pos0 = 8, 2, 128, 64, 512, 200
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, False)
    kp.copy_(rnd(kp.shape, 60).bfloat16())
    vp.copy_(rnd(vp.shape, 61).bfloat16())
    q = rnd((16, Hq * hd), 62, 0.5).bfloat16()
    full = torch.empty((16, Hq * hd), dtype=torch.bfloat16, device="cuda")
    B.ls_op_attention(q, pos0, Hq, Hkv, hd, page_size, table_d, max_seq, kp, vp, full)
    for m in (0, 3, 15):
        one = torch.empty((1, Hq * hd), dtype=torch.bfloat16, device="cuda")
        B.ls_op_attention(q[m:m + 1].contiguous(), pos0 + m, Hq, Hkv, hd, page_size, table_d, max_seq, kp, vp,
                          one)
        torch.cuda.synchronize()
        assert torch.equal(one[0], full[m]), f"row {m}"


# ------------------------------------------------------------------ accept / rollback
@pytest.mark.parametrize("draft,verified,max_new,eos,n_out0", [
    ([5, 6, 7], [9, 6, 7, 1], 10, -1, 0),
    ([5, 6, 7], [5, 6, 2, 1], 10, -1, 4),
    ([5, 6, 7], [5, 6, 7, 1], 10, -1, 0),
    ([5, 6, 7], [5, 6, 7, 1], 6, -1, 4),     # truncated at max_new: emits 2 of 4
    ([5, 6, 7], [5, 6, 7, 1], 10, 6, 0),     # EOS inside the accepted prefix
    ([], [3], 10, -1, 2),                    # d = 0: plain greedy bookkeeping
])
def test_accept_matches_oracle_match_and_bookkeeping(draft, verified, max_new, eos, n_out0):
    d = len(draft)
    dr = torch.tensor(draft + [0] * (16 - d), dtype=torch.int32, device="cuda")
    ve = torch.tensor(verified + [0] * (16 - len(verified)), dtype=torch.int32, device="cuda")
    state = torch.tensor([100, 42, n_out0, 3, 0, max_new, eos, 0], dtype=torch.int32, device="cuda")
    out = torch.full((32,), -1, dtype=torch.int32, device="cuda")
    acc = torch.full((32,), -1, dtype=torch.int32, device="cuda")
    B.ls_op_accept(dr, ve, d, state, out, acc)
    torch.cuda.synchronize()
    n = O.match(draft, verified[:d]) if d else 0
    emitted, stop = [], False
    for t in draft[:n] + [verified[n]]:
        if n_out0 + len(emitted) < max_new and not stop:
            emitted.append(t)
            stop = eos >= 0 and t == eos
    st = state.tolist()
    assert st[0] == 100 + n + 1 and st[1] == verified[n] and st[2] == n_out0 + len(emitted) and st[3] == 4
    assert st[4] == int(stop or st[2] >= max_new)
    assert out[n_out0:n_out0 + len(emitted)].tolist() == emitted and int(out[n_out0 + len(emitted)]) == -1
    assert int(acc[3]) == n
    # a finished loop is left alone
    if st[4]:
        B.ls_op_accept(dr, ve, d, state, out, acc)
        torch.cuda.synchronize()
        assert state.tolist() == st


def test_argument_errors_are_reported_not_launched():
    w = torch.zeros((16, 12), dtype=torch.bfloat16, device="cuda")  # K not a multiple of 8
    h = torch.zeros((1, 12), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(B.LsError) as e:
        B.ls_op_linear(B.LS_LINEAR_MMA, w, h, out)
    assert e.value.status == B.LS_ERR_INVALID_ARG
    w = torch.zeros((16, 16), dtype=torch.bfloat16, device="cuda")
    h = torch.zeros((17, 16), dtype=torch.bfloat16, device="cuda")  # too many rows
    with pytest.raises(B.LsError):
        B.ls_op_linear(B.LS_LINEAR_FMA, w, h, torch.zeros((17, 16), dtype=torch.float32, device="cuda"))
    with pytest.raises(B.LsError):
        B.ls_op_linear(3, w, h[:1].contiguous(), out)


# ------------------------------------------------------------------ prompt pass: tcgen05 GEMM, causal attention
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (31, 256, 256), (200, 688, 256), (512, 4096, 4096), (300, 1024, 11008),
                                   (130, 100, 72)])
@pytest.mark.parametrize("accumulate", [False, True])
def test_gemm_tensor_core(M, N, K, accumulate):
    a = rnd((M, K), 90).bfloat16()
    b = rnd((N, K), 91, 0.05).bfloat16()
    c = rnd((M, N), 92) if accumulate else torch.full((M, N), float("nan"), device="cuda")
    base = c.clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ls_op_gemm(a, b, c, accumulate, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0, "a bounded wait inside the GEMM ran out"
    rows = np.unique(np.concatenate([[0, M - 1, min(M - 1, 127), min(M - 1, 128)],
                                     np.random.default_rng(2).integers(0, M, 6)]))
    bb = bits(b)
    got = c.cpu().numpy().astype(np.float64)
    for m in rows:
        ref = O.linear(bb, vals(a[m])) + (base[m].cpu().numpy() if accumulate else 0.0)
        np.testing.assert_allclose(got[m], ref, rtol=0, atol=2e-5 * np.abs(ref).max() + 1e-6)
    assert np.isfinite(got).all()


# groups of 1, 2 and 4 query heads per KV head take the tensor-core kernel, 8 the FMA walk
@pytest.mark.parametrize("Hq,Hkv,hd", [(4, 2, 64), (4, 4, 128), (8, 2, 128), (8, 1, 64), (8, 1, 128)])
@pytest.mark.parametrize("R,pos0", [(1, 0), (16, 0), (37, 0), (100, 0), (50, 70)])
def test_prefill_attention(Hq, Hkv, hd, R, pos0):
    page_size, max_seq = 32, 256
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, True)
    n = pos0 + R
    kl = rnd((n + 8, Hkv, hd), 50).bfloat16()
    vl = rnd((n + 8, Hkv, hd), 51).bfloat16()
    for p in range(n + 8):
        kp[table[p // page_size], :, p % page_size, :] = kl[p]
        vp[table[p // page_size], :, p % page_size, :] = vl[p]
    q = rnd((R, Hq * hd), 52, 0.5).bfloat16()
    out = torch.empty((R, Hq * hd), dtype=torch.bfloat16, device="cuda")
    B.ls_op_prefill_attention(q, pos0, Hq, Hkv, hd, page_size, table_d, max_seq, kp, vp, out)
    torch.cuda.synchronize()
    kf, vf, qf = vals(kl).reshape(n + 8, -1), vals(vl).reshape(n + 8, -1), vals(q)
    for m in sorted({0, R // 2, R - 1, min(R - 1, 15), min(R - 1, 16)}):
        ref = O.attention(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd)
        assert (np.abs(vals(out[m]) - ref) <= attention_tol(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd, ref)).all()


# head dim 128 and at least 128 rows: the tcgen05 kernel (tiles of 128 rows, key blocks of 128).
# Pages smaller than, equal to and larger than a key block; row counts and start positions that
# leave ragged tiles and blocks; everything beyond the prompt holds NaN bit patterns, which must
# not reach any output.  ramp: keys grow with their position and the queries are large, so that
# a row's maximum keeps rising by more than the rescaling threshold from block to block.
@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2), (8, 1)])
@pytest.mark.parametrize("R,pos0,page_size,ramp", [(128, 0, 64, False), (200, 0, 16, False), (300, 77, 32, True),
                                                   (257, 1024, 256, False), (640, 130, 64, True), (129, 383, 128, False)])
def test_prefill_attention_tensor_core(Hq, Hkv, R, pos0, page_size, ramp):
    hd = 128
    n = pos0 + R
    max_seq = -(-(n + 130) // page_size) * page_size
    table, table_d, kp, vp = kv_setup(Hkv, hd, page_size, max_seq, True)
    kp.fill_(float("nan"))
    vp.fill_(float("nan"))
    kl = rnd((n, Hkv, hd), 60)
    if ramp:
        kl = kl * (1.0 + 3.0 * torch.arange(n, device="cuda").float() / n)[:, None, None]
    kl = kl.bfloat16()
    vl = rnd((n, Hkv, hd), 61).bfloat16()
    phys = torch.from_numpy(table[np.arange(n) // page_size].astype(np.int64)).cuda()
    slot = torch.arange(n, device="cuda") % page_size
    kp[phys, :, slot, :] = kl
    vp[phys, :, slot, :] = vl
    q = rnd((R, Hq * hd), 62, 3.0 if ramp else 0.5).bfloat16()
    out = torch.full((R, Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ls_op_prefill_attention(q, pos0, Hq, Hkv, hd, page_size, table_d, max_seq, kp, vp, out, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0, "a bounded wait inside the attention kernel ran out"
    assert torch.isfinite(out.float()).all()
    kf, vf, qf = vals(kl).reshape(n, -1), vals(vl).reshape(n, -1), vals(q)
    rows = sorted({0, 1, 127, 128 % R, R // 2, R - 1, (R - 1) // 128 * 128} | set(np.random.default_rng(4).integers(0, R, 4).tolist()))
    for m in rows:
        ref = O.attention(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd)
        assert (np.abs(vals(out[m]) - ref) <= attention_tol(qf[m], kf[:pos0 + m + 1], vf[:pos0 + m + 1], Hq, Hkv, hd, ref)).all(), m



def _tc_attention(q, kl, vl, pos0, Hq, Hkv, page_size, shuffle_seed):
    """ls_op_prefill_attention (head dim 128) of rows q at pos0 over the logical cache kl, vl laid out
    in pages of page_size tokens, permuted by shuffle_seed"""
    hd, n = 128, kl.shape[0]
    n_pages = -(-(n + 130) // page_size)
    table = np.random.default_rng(shuffle_seed).permutation(n_pages).astype(np.int32)
    kp = torch.full((n_pages, Hkv, page_size, hd), float("nan"), dtype=torch.bfloat16, device="cuda")
    vp = torch.full_like(kp, float("nan"))
    phys = torch.from_numpy(table[np.arange(n) // page_size].astype(np.int64)).cuda()
    slot = torch.arange(n, device="cuda") % page_size
    kp[phys, :, slot, :] = kl
    vp[phys, :, slot, :] = vl
    out = torch.full((q.shape[0], Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ls_op_prefill_attention(q, pos0, Hq, Hkv, hd, page_size, torch.from_numpy(table).cuda(), n_pages * page_size, kp, vp,
                              out, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    return out


def test_prefill_attention_tensor_core_depends_on_positions_only():
    """The tcgen05 kernel walks the cache by absolute position: the same logical cache in pages of 16,
    64 or 256 tokens, in any page order, gives the same bits; and rows 256.. of a prompt come out the
    same whether they are the tail of one call or a call of their own that starts at position 256
    (tiles of 128 rows and key blocks of 64 fall on the same positions)."""
    Hq, Hkv, hd, R = 8, 2, 128, 600
    kl = rnd((R, Hkv, hd), 70).bfloat16()
    vl = rnd((R, Hkv, hd), 71).bfloat16()
    q = rnd((R, Hq * hd), 72, 1.5).bfloat16()
    ref = _tc_attention(q, kl, vl, 0, Hq, Hkv, 64, 1)
    assert torch.isfinite(ref.float()).all()
    for page_size, seed in ((16, 2), (256, 3), (64, 4)):
        assert torch.equal(_tc_attention(q, kl, vl, 0, Hq, Hkv, page_size, seed), ref), page_size
    tail = _tc_attention(q[256:].contiguous(), kl, vl, 256, Hq, Hkv, 32, 5)
    assert torch.equal(tail, ref[256:])
