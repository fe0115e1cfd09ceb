"""The calls on either side of an exchange between GPUs, against the CPU oracle, bit for bit.

s3gd_vote_apply (vote over a message gathered from several senders, fused with the update),
s3gd_vote_counts (vote sums that add up across GPUs), s3gd_encode_vote2 / s3gd_apply_vote2 (the
server's message in two bits per coordinate), s3gd_encode_vote_sparse / s3gd_apply_vote_sparse (the
same message as a list of coordinates and sign bits).  Everything is integer work or one fp32 rounding:
tolerance 0.  The exchange itself is emulated on one GPU by laying the senders' pieces side by side,
which is exactly what an all-gather produces, and by adding the senders' sums as a reduce-scatter would.
"""
import numpy as np
import pytest
import torch

import paper_2302_07475_b200 as S
from oracle import s3gd_oracle as O
from paper_2302_07475_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _pieces(grads, n_groups, K, pad_words):
    """TopKSign of each group's rows written into one buffer, pieces `stride` words apart."""
    M, d = grads.shape
    Mg = M // n_groups
    Wd = S.binding.words(K)
    stride = Mg * (K + Wd) + pad_words
    msg = torch.full((n_groups * stride,), -1, dtype=torch.int32, device=DEV)
    ws = S.alloc_workspace(Mg, d, K, DEV)
    for g in range(n_groups):
        piece = msg[g * stride: g * stride + Mg * (K + Wd)]
        S.s3gd_topk_sign(grads[g * Mg:(g + 1) * Mg].contiguous(), K, piece[:Mg * K].view(Mg, K), piece[Mg * K:].view(Mg, Wd), ws)
    S.s3gd_device_status(ws)
    return msg, stride, Mg


@pytest.mark.parametrize("M,n_groups,d,K,pad", [(6, 2, 300_007, 3_000, 0), (6, 3, 300_007, 300, 5), (8, 1, 40_001, 10_000, 0),
                                                (130, 2, 20_003, 500, 3), (127, 1, 20_003, 20_003, 0), (4, 4, 1_000, 0, 2)])
def test_vote_apply_over_a_gathered_message(M, n_groups, d, K, pad):
    s = W.spec("resnet18", d=d, M=M)
    g, x = W.make_grads(s, DEV), W.make_x(s, DEV)
    g[:, 7] = 1e3
    g[:, d - 2] = -1e3                                  # unanimous votes: the counts reach +M and -M
    x_o, idx_o, sgn_o, vote_o = O.step(x.cpu().numpy(), g.cpu().numpy(), K, s.lr)
    msg, stride, Mg = _pieces(g, n_groups, K, pad)
    ws = S.alloc_workspace(M, d, K, DEV)
    ws.fill_(0x77)
    vote = torch.full((d,), 55, dtype=torch.int8, device=DEV)
    xa = x.clone()
    S.s3gd_vote_apply(xa, msg, n_groups, stride, Mg, K, s.lr, ws, vote)
    code, info = S.s3gd_device_status(ws)
    assert code == 0 and info[2] == 0
    assert np.array_equal(vote.cpu().numpy(), vote_o)
    assert np.array_equal(bits(xa.cpu().numpy()), bits(x_o))
    xb = x.clone()                                      # without the optional vote
    S.s3gd_vote_apply(xb, msg, n_groups, stride, Mg, K, s.lr, ws)
    S.s3gd_device_status(ws)
    assert np.array_equal(bits(xb.cpu().numpy()), bits(x_o))


def test_vote_apply_flags_an_index_out_of_range():
    d, M, K = 1000, 3, 8
    s = W.spec("tiny", d=d, M=M)
    g, x = W.make_grads(s, DEV), W.make_x(s, DEV)
    msg, stride, Mg = _pieces(g, 1, K, 0)
    msg[5] = d + 3
    idx = u32(msg[:M * K]).reshape(M, K)
    sgn = u32(msg[M * K:M * K + M]).reshape(M, 1)
    vote_o, bad = O.majority_vote(idx, sgn, M, K, d)
    assert bad == 1
    ws = S.alloc_workspace(M, d, K, DEV)
    vote = torch.empty(d, dtype=torch.int8, device=DEV)
    S.s3gd_vote_apply(x, msg, 1, stride, Mg, K, s.lr, ws, vote)
    code, info = S.s3gd_device_status(ws, raise_on_error=False)
    assert code == 4 and info[2] == 1 and np.array_equal(vote.cpu().numpy(), vote_o)


@pytest.mark.parametrize("M,d,K,senders", [(6, 100_003, 2_000, 2), (90, 30_001, 700, 3), (140, 30_001, 700, 2), (5, 17, 17, 5)])
def test_vote_counts_add_up_across_senders_and_encode_to_two_bits(M, d, K, senders):
    s = W.spec("small_cnn", d=d, M=M)
    g, x = W.make_grads(s, DEV), W.make_x(s, DEV)
    g[:, 3] = 77.0                                      # every worker votes +1 here
    gn = g.cpu().numpy()
    idx_o, sgn_o = O.topk_sign_threshold(gn, K)
    vote_o, _ = O.majority_vote(idx_o, sgn_o, M, K, d)
    x_o = O.apply_vote(x.cpu().numpy(), vote_o, s.lr)
    Ms = M // senders
    d_pad = (d + 63) // 64 * 64
    as_bytes = M <= 127
    dtype = torch.uint8 if as_bytes else torch.int32
    ws = S.alloc_workspace(Ms, d, K, DEV)
    total = torch.zeros(d_pad, dtype=torch.int64, device=DEV)
    for r in range(senders):
        rows = g[r * Ms:(r + 1) * Ms].contiguous()
        idx = torch.empty((Ms, K), dtype=torch.int32, device=DEV)
        sgn = torch.empty((Ms, S.binding.words(K)), dtype=torch.int32, device=DEV)
        S.s3gd_topk_sign(rows, K, idx, sgn, ws)
        counts = torch.full((d_pad,), 9, dtype=dtype, device=DEV)
        bad = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        S.s3gd_vote_counts(idx, sgn, Ms, K, d, counts, bad)
        torch.cuda.synchronize()
        want = np.zeros(d_pad, np.int64)
        want[:d] = O.vote_counts(idx_o[r * Ms:(r + 1) * Ms], sgn_o[r * Ms:(r + 1) * Ms], Ms, K, d)
        got = counts.cpu().numpy().astype(np.int64) - (128 if as_bytes else 0)
        assert np.array_equal(got, want) and int(bad.item()) == 0, f"sender {r}"
        total += counts.to(torch.int64)
    summed = (total % 256).to(torch.uint8) if as_bytes else total.to(torch.int32)     # what a sum-reduce delivers
    words2 = torch.full(((d_pad + 15) // 16,), -1, dtype=torch.int32, device=DEV)
    S.s3gd_encode_vote2(summed, words2, n_summed=senders)
    torch.cuda.synchronize()
    pad_vote = np.zeros(d_pad, np.int8)
    pad_vote[:d] = vote_o
    assert np.array_equal(u32(words2), O.encode_vote_2bit(pad_vote))
    vote = torch.full((d,), 33, dtype=torch.int8, device=DEV)
    xa = x.clone()
    S.s3gd_apply_vote2(xa, words2, s.lr, vote)
    torch.cuda.synchronize()
    assert np.array_equal(vote.cpu().numpy(), vote_o) and np.array_equal(bits(xa.cpu().numpy()), bits(x_o))
    xb = x.clone()
    S.s3gd_apply_vote2(xb, words2, s.lr)
    torch.cuda.synchronize()
    assert np.array_equal(bits(xb.cpu().numpy()), bits(x_o))


@pytest.mark.parametrize("d", [1, 15, 16, 17, 1_000_003])
def test_two_bit_form_of_an_int8_vote(d):
    gen = torch.Generator(DEV).manual_seed(d)
    vote = torch.randint(-1, 2, (d,), generator=gen, device=DEV, dtype=torch.int8)
    words2 = torch.full(((d + 15) // 16,), -1, dtype=torch.int32, device=DEV)
    S.s3gd_encode_vote2(vote, words2)
    torch.cuda.synchronize()
    assert np.array_equal(u32(words2), O.encode_vote_2bit(vote.cpu().numpy()))
    # apply leaves unvoted bits alone, NaN payloads and signed zeros included
    xb = np.resize(np.array([0x7FC12345, 0x80000000, 0x00000001, 0x3F800000, 0x7F800000, 0x3DCCCCCD], np.uint32), d)
    x = torch.from_numpy(xb.view(np.float32).copy()).to(DEV)
    back = torch.empty(d, dtype=torch.int8, device=DEV)
    S.s3gd_apply_vote2(x, words2, 0.3, back)
    torch.cuda.synchronize()
    want = O.apply_vote(xb.view(np.float32), O.decode_vote_2bit(O.encode_vote_2bit(vote.cpu().numpy()), d), 0.3)
    got = x.cpu().numpy()
    assert np.all((bits(got) == bits(want)) | (np.isnan(got) & np.isnan(want)))
    v = vote.cpu().numpy()
    assert np.array_equal(bits(got)[v == 0], xb[v == 0]) and np.array_equal(back.cpu().numpy(), v)


def _sparse_piece(vote_np, cap, index_base=0):
    """The oracle's sparse form laid out as the library's piece: count, cap indices, sign words."""
    idx, sgn = O.encode_vote_sparse(vote_np)
    piece = np.zeros(S.binding.sparse_piece_words(cap), np.uint32)
    piece[0] = idx.shape[0]
    n = min(idx.shape[0], cap)
    piece[1:1 + n] = idx[:n] + np.uint32(index_base)
    full = O.pack_sign_bits(vote_np[idx[:n].astype(np.int64)] < 0) if n else np.zeros(0, np.uint32)
    piece[1 + cap:1 + cap + full.shape[0]] = full
    return piece


def _same_piece(got, want, cap):
    """Count, the listed indices and every sign word must agree; index slots beyond the count are unspecified."""
    n = min(int(want[0]), cap)
    return got[0] == want[0] and np.array_equal(got[1:1 + n], want[1:1 + n]) and np.array_equal(got[1 + cap:], want[1 + cap:])


@pytest.mark.parametrize("d,density,cap", [(1, 1.0, 4), (4095, 0.3, 4095), (4097, 0.02, 200), (100_003, 0.05, 6_000),
                                           (100_003, 0.5, 1_000), (1_000_003, 0.001, 2_048)])
def test_sparse_form_of_the_vote(d, density, cap):
    gen = torch.Generator(DEV).manual_seed(d + cap)
    moved = torch.rand(d, generator=gen, device=DEV) < density
    sign = torch.where(torch.rand(d, generator=gen, device=DEV) < 0.5, -1, 1).to(torch.int8)
    vote = torch.where(moved, sign, torch.zeros_like(sign))
    v = vote.cpu().numpy()
    ws = torch.empty(max(S.s3gd_sparse_workspace_bytes(d), 4), dtype=torch.uint8, device=DEV)
    for src, n_summed in ((vote, 1), (vote.to(torch.int32) * 3, 1),
                          (((vote.to(torch.int64) * 2 + 128 * 3) % 256).to(torch.uint8), 3)):     # int8 votes, int32 sums, summed bytes
        piece = torch.full((S.binding.sparse_piece_words(cap),), -1, dtype=torch.int32, device=DEV)
        S.s3gd_encode_vote_sparse(src, piece, cap, ws, index_base=0, n_summed=n_summed)
        torch.cuda.synchronize()
        assert _same_piece(u32(piece), _sparse_piece(v, cap), cap), f"source {src.dtype}"
    # a range that does not start at coordinate 0, applied next to a second piece for the coordinates before it
    half = d // 2
    lo_piece = torch.from_numpy(_sparse_piece(v[:half], cap).view(np.int32).copy()).to(DEV) if half else None
    hi_piece = torch.empty(S.binding.sparse_piece_words(cap), dtype=torch.int32, device=DEV)
    S.s3gd_encode_vote_sparse(vote[half:].contiguous(), hi_piece, cap, ws, index_base=half)
    torch.cuda.synchronize()
    assert _same_piece(u32(hi_piece), _sparse_piece(v[half:], cap, index_base=half), cap)
    if half and np.count_nonzero(v[:half]) <= cap and np.count_nonzero(v[half:]) <= cap:
        stride = S.binding.sparse_piece_words(cap) + 3
        both = torch.zeros(2 * stride, dtype=torch.int32, device=DEV)
        both[:lo_piece.numel()] = lo_piece
        both[stride:stride + hi_piece.numel()] = hi_piece
        x = torch.linspace(-1, 1, d, device=DEV)
        x_o = O.apply_vote(x.cpu().numpy(), v, 0.125)
        bad = torch.full((1,), -1, dtype=torch.int32, device=DEV)
        S.s3gd_apply_vote_sparse(x, both, 2, stride, cap, 0.125, bad)
        torch.cuda.synchronize()
        assert np.array_equal(bits(x.cpu().numpy()), bits(x_o)) and int(bad.item()) == 0


def test_sparse_apply_skips_an_index_out_of_range():
    d, cap = 50, 8
    piece = np.zeros(S.binding.sparse_piece_words(cap), np.uint32)
    piece[0] = 3
    piece[1:4] = [2, 49, 50]
    piece[1 + cap] = 0b010
    x = torch.zeros(d, device=DEV)
    bad = torch.zeros(1, dtype=torch.int32, device=DEV)
    S.s3gd_apply_vote_sparse(x, torch.from_numpy(piece.view(np.int32).copy()).to(DEV), 1, piece.shape[0], cap, 0.5, bad)
    torch.cuda.synchronize()
    want = np.zeros(d, np.float32)
    want[2], want[49] = -0.5, 0.5
    assert np.array_equal(x.cpu().numpy(), want) and int(bad.item()) == 1
