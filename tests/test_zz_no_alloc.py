"""The allocation-free majority vote against the ordinary one (collected last on purpose).

s3gd_majority_vote_noalloc exists for callers that cannot get device memory at the place
where they vote: code inside another framework's callback that must stay out of that
framework's allocator, plug-ins that only ever see their input and output buffers, or a
process whose GPU memory already belongs to a pool it does not own.  Its counters are a
fixed array inside the library, shared by every call, so the interesting failure is a
second call that sees what the first one left behind.  The test therefore makes two calls
in a row -- the second on a different, much sparser message -- and requires each result to
equal s3gd_majority_vote's on the same inputs exactly (votes are integers: tolerance 0), and
both to equal the CPU oracle's vote, so that a mistake the two library calls share (they use the
same two kernels) cannot hide.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2302_07475_b200 as S
from oracle import s3gd_oracle as O

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _message(M, K, d, seed):
    g = torch.Generator(DEV).manual_seed(seed)
    idx = torch.randint(0, d, (M, K), generator=g, device=DEV, dtype=torch.int32)
    sgn = torch.randint(-2**31, 2**31 - 1, (M, (K + 31) // 32), generator=g, device=DEV, dtype=torch.int64).to(torch.int32)
    return idx.contiguous(), sgn.contiguous()


def _both(idx, sgn, M, K, d):
    ref = torch.full((d,), 55, dtype=torch.int8, device=DEV)
    ws = S.alloc_workspace(M, d, K, DEV)
    S.s3gd_majority_vote(idx, sgn, M, K, d, ref, ws)
    S.s3gd_device_status(ws, raise_on_error=False)
    got = torch.full((d,), 66, dtype=torch.int8, device=DEV)
    bad = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    S.s3gd_majority_vote_noalloc(idx, sgn, M, K, d, got, bad)
    torch.cuda.synchronize()
    want, want_bad = O.majority_vote(idx.cpu().numpy().view(np.uint32), sgn.cpu().numpy().view(np.uint32), M, K, d)
    assert np.array_equal(got.cpu().numpy(), want) and int(bad.item()) == want_bad, "differs from the oracle's vote"
    return ref.cpu().numpy(), got.cpu().numpy(), int(bad.item())


def test_two_calls_in_a_row_match_the_ordinary_vote():
    d = 1_000_003
    assert d <= S.s3gd_noalloc_max_d()
    # first call: dense message, most coordinates get votes
    M, K = 9, 400_000
    idx, sgn = _message(M, K, d, seed=1)
    ref, got, bad = _both(idx, sgn, M, K, d)
    assert np.array_equal(ref, got) and bad == 0
    assert np.count_nonzero(ref) > d // 2
    # second call: a sparse message on a shorter vector; stale counters from the first
    # call, inside or beyond the new d, would show up as wrong votes
    M2, K2, d2 = 3, 1_000, 700_001
    idx2, sgn2 = _message(M2, K2, d2, seed=2)
    idx2[1, 7] = d2 + 5                      # one index out of range: skipped and counted
    ref2, got2, bad2 = _both(idx2, sgn2, M2, K2, d2)
    assert np.array_equal(ref2, got2) and bad2 == 1
    assert np.count_nonzero(ref2) <= M2 * K2


def test_rejects_more_coordinates_than_the_built_in_counters_hold():
    lib = S.load()
    fake = ctypes.c_void_p(4096)             # never dereferenced: the size check comes first
    too_many = S.s3gd_noalloc_max_d() + 1
    assert lib.s3gd_majority_vote_noalloc(fake, fake, 1, 1, too_many, fake, None, None) == 6
    assert S.s3gd_status_string(6) == "S3GD_ERR_TOO_LARGE"
