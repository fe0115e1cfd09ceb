"""Host-side checks that need no GPU: the library loads, exports what the header
declares, sizes workspaces sanely and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

import paper_2302_07475_b200 as S
from paper_2302_07475_b200 import binding, build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return binding.load()


def test_exports_match_header(lib):
    with open(os.path.join(ROOT, "include", "s3gd.h")) as f:
        text = f.read()
    declared = set(re.findall(r"S3GD_API[^;(]*?\b(s3gd_\w+)\s*\(", text))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for code, name in binding.STATUS_NAMES.items():
        assert S.s3gd_status_string(code) == name
    assert S.s3gd_status_string(99) == "S3GD_ERR_UNKNOWN"


def test_workspace_bytes(lib):
    assert S.s3gd_workspace_bytes(0, 10, 1) == 0          # M <= 0
    assert S.s3gd_workspace_bytes(1, 0, 0) == 0           # d == 0
    assert S.s3gd_workspace_bytes(1, 1 << 32, 1) == 0     # d does not fit uint32 indices
    assert S.s3gd_workspace_bytes(1, 10, 11) == 0         # K > d
    small = S.s3gd_workspace_bytes(5, 65536, 655)
    assert small >= 65536 * 4 and small % 256 == 0
    # the counters dominate for small K; the size grows with K and with d
    a = S.s3gd_workspace_bytes(32, 25_557_032, 2_556)
    b = S.s3gd_workspace_bytes(32, 25_557_032, 255_570)
    assert 25_557_032 * 4 <= a < b < 2 * 1024**3
    big = S.s3gd_workspace_bytes(8, 2_100_000_000, 2_100_000)
    assert 8.4e9 < big < 10e9                              # fits beside 67 GB of gradients and 8.4 GB of x


def test_bad_arguments_rejected_before_launch(lib):
    vp = ctypes.c_void_p
    fake = vp(256 * 1024)          # never dereferenced: every call below fails validation first
    INV, WS = 1, 2
    assert lib.s3gd_topk_sign(None, 1, 8, 2, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_topk_sign(fake, 0, 8, 2, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_topk_sign(fake, 1, 8, 9, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_topk_sign(fake, 1, 8, 2, None, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_topk_sign(fake, 1, 8, 2, fake, fake, None, 1 << 30, None) == WS
    assert lib.s3gd_topk_sign(fake, 1, 8, 2, fake, fake, fake, 16, None) == WS          # too small
    assert lib.s3gd_topk_sign(fake, 1, 8, 2, fake, fake, vp(256 * 1024 + 8), 1 << 30, None) == WS  # misaligned
    assert lib.s3gd_topk_sign(vp(256 * 1024 + 2), 1, 8, 2, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_majority_vote(None, fake, 1, 2, 8, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_majority_vote(fake, fake, 1, 2, 8, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_apply(None, fake, 8, 0.1, None) == INV
    assert lib.s3gd_apply(fake, None, 8, 0.1, None) == INV
    assert lib.s3gd_apply(fake, fake, 0, 0.1, None) == INV
    assert lib.s3gd_step(None, fake, 1, 8, 2, 0.1, None, None, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_step(fake, fake, 1, 8, 2, 0.1, fake, None, None, fake, 1 << 30, None) == INV  # idx without signs
    assert lib.s3gd_step(fake, fake, 1, 8, 2, 0.1, None, None, None, fake, 8, None) == WS
    assert lib.s3gd_device_status(None, None, None) == WS
    assert lib.s3gd_step_ex(None, fake, None, 1.0, None, 0.0, 1, 8, 2, 0.1, None, None, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_step_ex(fake, fake, vp(256 * 1024 + 1), 1.0, None, 0.0, 1, 8, 2, 0.1, None, None, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_apply_momentum(fake, None, fake, 8, 0.5, 0.1, None) == INV
    assert lib.s3gd_randk_sign(None, 1, 8, 2, 1, 0, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_randk_sign(fake, 1, 8, 9, 1, 0, fake, fake, fake, 1 << 30, None) == INV
    assert lib.s3gd_randk_sign(fake, 1, 8, 2, 1, 0, fake, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_randk_sign(fake, 1, 8, 2, 1, 0, fake, fake, fake, 8, None) == WS
    assert lib.s3gd_step_randk(None, fake, 1, 8, 2, 0.1, 1, 0, None, None, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_step_randk(fake, fake, 1, 8, 2, 0.1, 1, 0, fake, None, None, fake, 1 << 30, None) == INV
    assert lib.s3gd_step_randk(fake, fake, 1, 8, 2, 0.1, 1, 0, None, None, None, None, 1 << 30, None) == WS


def test_exchange_calls_reject_bad_arguments(lib):
    fake = ctypes.c_void_p(256 * 1024)
    assert lib.s3gd_vote_apply(fake, fake, 0, 10, 1, 2, 8, 0.1, None, fake, 1 << 30, None) == 1       # no groups
    assert lib.s3gd_vote_apply(fake, fake, 2, 1, 1, 2, 8, 0.1, None, fake, 1 << 30, None) == 1        # pieces overlap
    assert lib.s3gd_vote_apply(fake, fake, 2, 10, 1, 2, 8, 0.1, None, fake, 8, None) == 2             # workspace too small
    assert lib.s3gd_vote_counts(fake, fake, 200, 2, 8, 8, fake, 1, None, None) == 1                   # bytes cannot count 200 workers
    assert lib.s3gd_vote_counts(fake, fake, 2, 2, 8, 6, fake, 4, None, None) == 1                     # padded length below d
    assert lib.s3gd_vote_counts(fake, fake, 2, 2, 8, 8, fake, 2, None, None) == 1                     # counts are 1 or 4 bytes
    assert lib.s3gd_encode_vote2(fake, 3, 1, 8, fake, None) == 1
    assert lib.s3gd_apply_vote2(None, fake, 8, 0.1, None, None) == 1
    assert lib.s3gd_sparse_workspace_bytes(0) == 0 and lib.s3gd_sparse_workspace_bytes(4096) == 4
    assert lib.s3gd_sparse_workspace_bytes(4097) == 8
    assert lib.s3gd_encode_vote_sparse(fake, 2, 1, 8, 0, 0, fake, fake, 64, None) == 1               # no room at all
    assert lib.s3gd_encode_vote_sparse(fake, 2, 1, 8, 0, 4, fake, fake, 2, None) == 2                # scratch too small
    assert lib.s3gd_encode_vote_sparse(fake, 2, 1, 8, 0xFFFFFFFF, 4, fake, fake, 64, None) == 1      # coordinates past 2^32
    assert lib.s3gd_apply_vote_sparse(fake, fake, 2, 5, 8, 100, 0.1, None, None) == 1                # pieces overlap


def test_binding_refuses_cpu_tensors(lib):
    import torch
    g = torch.zeros((2, 64))
    with pytest.raises(TypeError):
        S.s3gd_step(torch.zeros(64), g, 4, 0.1, torch.zeros(1024, dtype=torch.uint8))


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        binding.load(str(tmp_path / "nope.so"))
