"""The calls on either side of an exchange between GPUs, against the CPU oracle, bit for bit.

s3gd_vote_apply (vote over a message gathered from several senders, fused with the update),
s3gd_vote_counts (vote sums that add up across GPUs), s3gd_encode_vote2 / s3gd_apply_vote2 (the
server's message in two bits per coordinate).  Everything is integer work or one fp32 rounding:
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
