"""ctypes binding of libs3gd.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the CUDA kernels of the library; nothing here
computes.  torch is used for device buffers and the current stream.  If the
library is missing or a tensor is not a contiguous CUDA tensor of the right
dtype the call raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# S3GD_LIBRARY names another build of the same library (same C ABI) to load instead of the in-tree one
LIB_PATH = os.environ.get("S3GD_LIBRARY") or os.path.join(_PKG, "libs3gd.so")

S3GD_OK = 0
STATUS_NAMES = {
    0: "S3GD_OK", 1: "S3GD_ERR_INVALID_ARG", 2: "S3GD_ERR_WORKSPACE", 3: "S3GD_ERR_CUDA",
    4: "S3GD_ERR_INDEX_RANGE", 5: "S3GD_ERR_INTERNAL", 6: "S3GD_ERR_TOO_LARGE",
}

EXPORTS = ("s3gd_status_string", "s3gd_workspace_bytes", "s3gd_topk_sign", "s3gd_majority_vote",
           "s3gd_apply", "s3gd_step", "s3gd_device_status", "s3gd_profile_begin", "s3gd_profile_end",
           "s3gd_noalloc_max_d", "s3gd_majority_vote_noalloc", "s3gd_step_ex", "s3gd_apply_momentum",
           "s3gd_randk_sign", "s3gd_step_randk", "s3gd_profile_begin_filter", "s3gd_last_device_status",
           "s3gd_debug_topk_sign", "s3gd_debug_step", "s3gd_vote_apply", "s3gd_vote_counts", "s3gd_encode_vote2",
           "s3gd_apply_vote2", "s3gd_sparse_workspace_bytes", "s3gd_encode_vote_sparse", "s3gd_apply_vote_sparse",
           "s3gd_profile_begin_filter_every")


class S3gdError(RuntimeError):
    def __init__(self, call: str, code: int):
        super().__init__(f"{call} returned {STATUS_NAMES.get(code, code)}")
        self.code = code


_lib = None


def load(path: Optional[str] = None) -> ctypes.CDLL:
    """Load the shared library (once) and declare the argument types of every export."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2302_07475_b200.build` (needs nvcc); "
            "there is no fallback implementation")
    lib = ctypes.CDLL(p)
    vp, u64, u32p, sz = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_size_t
    lib.s3gd_status_string.restype = ctypes.c_char_p
    lib.s3gd_status_string.argtypes = [ctypes.c_int]
    lib.s3gd_workspace_bytes.restype = sz
    lib.s3gd_workspace_bytes.argtypes = [ctypes.c_int, u64, u64]
    lib.s3gd_topk_sign.restype = ctypes.c_int
    lib.s3gd_topk_sign.argtypes = [vp, ctypes.c_int, u64, u64, u32p, u32p, vp, sz, vp]
    lib.s3gd_majority_vote.restype = ctypes.c_int
    lib.s3gd_majority_vote.argtypes = [u32p, u32p, ctypes.c_int, u64, u64, vp, vp, sz, vp]
    lib.s3gd_apply.restype = ctypes.c_int
    lib.s3gd_apply.argtypes = [vp, vp, u64, ctypes.c_float, vp]
    lib.s3gd_step.restype = ctypes.c_int
    lib.s3gd_step.argtypes = [vp, vp, ctypes.c_int, u64, u64, ctypes.c_float, u32p, u32p, vp, vp, sz, vp]
    lib.s3gd_device_status.restype = ctypes.c_int
    lib.s3gd_device_status.argtypes = [vp, vp, ctypes.c_void_p]
    lib.s3gd_profile_begin.restype = ctypes.c_int
    lib.s3gd_profile_begin.argtypes = [ctypes.c_int]
    lib.s3gd_profile_end.restype = ctypes.c_int
    lib.s3gd_profile_end.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.s3gd_noalloc_max_d.restype = ctypes.c_uint64
    lib.s3gd_noalloc_max_d.argtypes = []
    lib.s3gd_majority_vote_noalloc.restype = ctypes.c_int
    lib.s3gd_majority_vote_noalloc.argtypes = [u32p, u32p, ctypes.c_int, u64, u64, vp, vp, vp]
    lib.s3gd_step_ex.restype = ctypes.c_int
    lib.s3gd_step_ex.argtypes = [vp, vp, vp, ctypes.c_float, vp, ctypes.c_float, ctypes.c_int, u64, u64, ctypes.c_float,
                                 u32p, u32p, vp, vp, sz, vp]
    lib.s3gd_apply_momentum.restype = ctypes.c_int
    lib.s3gd_apply_momentum.argtypes = [vp, vp, vp, u64, ctypes.c_float, ctypes.c_float, vp]
    lib.s3gd_profile_begin_filter.restype = ctypes.c_int
    lib.s3gd_profile_begin_filter.argtypes = [ctypes.c_int]
    lib.s3gd_profile_begin_filter_every.restype = ctypes.c_int
    lib.s3gd_profile_begin_filter_every.argtypes = [ctypes.c_int, ctypes.c_int]
    u32 = ctypes.c_uint32
    lib.s3gd_randk_sign.restype = ctypes.c_int
    lib.s3gd_randk_sign.argtypes = [vp, ctypes.c_int, u64, u64, u32, u32, u32p, u32p, vp, sz, vp]
    lib.s3gd_step_randk.restype = ctypes.c_int
    lib.s3gd_step_randk.argtypes = [vp, vp, ctypes.c_int, u64, u64, ctypes.c_float, u32, u32, u32p, u32p, vp, vp, sz, vp]
    lib.s3gd_last_device_status.restype = ctypes.c_int
    lib.s3gd_last_device_status.argtypes = [vp, vp]
    lib.s3gd_debug_topk_sign.restype = ctypes.c_int
    lib.s3gd_debug_topk_sign.argtypes = lib.s3gd_topk_sign.argtypes + [u32]
    lib.s3gd_debug_step.restype = ctypes.c_int
    lib.s3gd_debug_step.argtypes = lib.s3gd_step.argtypes + [u32, u32]
    lib.s3gd_vote_apply.restype = ctypes.c_int
    lib.s3gd_vote_apply.argtypes = [vp, u32p, ctypes.c_int, u64, ctypes.c_int, u64, u64, ctypes.c_float, vp, vp, sz, vp]
    lib.s3gd_vote_counts.restype = ctypes.c_int
    lib.s3gd_vote_counts.argtypes = [u32p, u32p, ctypes.c_int, u64, u64, u64, vp, ctypes.c_int, vp, vp]
    lib.s3gd_encode_vote2.restype = ctypes.c_int
    lib.s3gd_encode_vote2.argtypes = [vp, ctypes.c_int, u32, u64, u32p, vp]
    lib.s3gd_apply_vote2.restype = ctypes.c_int
    lib.s3gd_apply_vote2.argtypes = [vp, u32p, u64, ctypes.c_float, vp, vp]
    lib.s3gd_sparse_workspace_bytes.restype = sz
    lib.s3gd_sparse_workspace_bytes.argtypes = [u64]
    lib.s3gd_encode_vote_sparse.restype = ctypes.c_int
    lib.s3gd_encode_vote_sparse.argtypes = [vp, ctypes.c_int, u32, u64, u32, u32, u32p, vp, sz, vp]
    lib.s3gd_apply_vote_sparse.restype = ctypes.c_int
    lib.s3gd_apply_vote_sparse.argtypes = [vp, u32p, ctypes.c_int, u64, u32, u64, ctypes.c_float, vp, vp]
    if path is None:
        _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, numel: Optional[int] = None, name: str = "tensor"):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    if numel is not None and t.numel() < numel:
        raise ValueError(f"{name} has {t.numel()} elements, needs {numel}")
    return ctypes.c_void_p(t.data_ptr())


def _stream(t: torch.Tensor):
    return ctypes.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _check(call: str, code: int) -> None:
    if code != S3GD_OK:
        raise S3gdError(call, code)


def s3gd_status_string(code: int) -> str:
    return load().s3gd_status_string(int(code)).decode()


def s3gd_workspace_bytes(M: int, d: int, K: int) -> int:
    return int(load().s3gd_workspace_bytes(int(M), int(d), int(K)))


def alloc_workspace(M: int, d: int, K: int, device="cuda") -> torch.Tensor:
    """A uint8 CUDA tensor of s3gd_workspace_bytes(M, d, K) bytes (torch allocations are 512-byte aligned)."""
    n = s3gd_workspace_bytes(M, d, K)
    if n == 0:
        raise ValueError("invalid (M, d, K)")
    return torch.empty(n, dtype=torch.uint8, device=device)


def words(K: int) -> int:
    return (int(K) + 31) // 32


def s3gd_topk_sign(grads: torch.Tensor, K: int, out_idx: torch.Tensor, out_signbits: torch.Tensor,
                   ws: torch.Tensor) -> None:
    """grads [M, d] fp32 -> out_idx [M, K] (uint32 values in int32 storage), out_signbits [M, ceil(K/32)]."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (g, M, d, K, _ptr(out_idx, torch.int32, M * K, "out_idx"),
            _ptr(out_signbits, torch.int32, M * words(K), "out_signbits"),
            _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(grads.device):
        code = load().s3gd_topk_sign(*args, _stream(grads))
    _check("s3gd_topk_sign", code)


def s3gd_majority_vote(idx: torch.Tensor, signbits: torch.Tensor, M: int, K: int, d: int,
                       out_vote: torch.Tensor, ws: torch.Tensor) -> None:
    """idx [M, K], signbits [M, ceil(K/32)] -> out_vote [d] int8 in {-1, 0, +1}."""
    args = (_ptr(idx, torch.int32, M * K, "idx"), _ptr(signbits, torch.int32, M * words(K), "signbits"), M, K, d,
            _ptr(out_vote, torch.int8, d, "out_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(out_vote.device):
        code = load().s3gd_majority_vote(*args, _stream(out_vote))
    _check("s3gd_majority_vote", code)


def s3gd_apply(x: torch.Tensor, vote: torch.Tensor, lr: float) -> None:
    """x [d] fp32 updated in place by -lr * vote."""
    d = x.numel()
    args = (_ptr(x, torch.float32, name="x"), _ptr(vote, torch.int8, d, "vote"), d, ctypes.c_float(lr))
    with torch.cuda.device(x.device):
        code = load().s3gd_apply(*args, _stream(x))
    _check("s3gd_apply", code)


def s3gd_step(x: torch.Tensor, grads: torch.Tensor, K: int, lr: float, ws: torch.Tensor,
              opt_idx: Optional[torch.Tensor] = None, opt_signbits: Optional[torch.Tensor] = None,
              opt_vote: Optional[torch.Tensor] = None) -> None:
    """The fused step: x [d] updated in place from grads [M, d]; optional outputs as in the unfused calls."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (_ptr(x, torch.float32, d, "x"), g, M, d, K, ctypes.c_float(lr),
            _ptr(opt_idx, torch.int32, M * K, "opt_idx"), _ptr(opt_signbits, torch.int32, M * words(K), "opt_signbits"),
            _ptr(opt_vote, torch.int8, d, "opt_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(x.device):
        code = load().s3gd_step(*args, _stream(x))
    _check("s3gd_step", code)


def s3gd_device_status(ws: torch.Tensor, raise_on_error: bool = True):
    """Synchronises the current stream; returns (status code, 8 diagnostic counters)."""
    info = (ctypes.c_uint32 * 8)()
    w = _ptr(ws, torch.uint8, name="ws")
    with torch.cuda.device(ws.device):
        code = load().s3gd_device_status(w, _stream(ws), info)
    if raise_on_error:
        _check("s3gd_device_status", code)
    return code, list(info)


def s3gd_last_device_status(ws: torch.Tensor) -> int:
    """Synchronises the current stream; returns the status code recorded by the kernels (0 = ok)."""
    w = _ptr(ws, torch.uint8, name="ws")
    with torch.cuda.device(ws.device):
        return int(load().s3gd_last_device_status(w, _stream(ws)))


def s3gd_debug_topk_sign(grads: torch.Tensor, K: int, out_idx: torch.Tensor, out_signbits: torch.Tensor,
                         ws: torch.Tensor, sample_rank: int) -> None:
    """s3gd_topk_sign with the sampling rank of the filter threshold forced (0: the library's own)."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (g, M, d, K, _ptr(out_idx, torch.int32, M * K, "out_idx"),
            _ptr(out_signbits, torch.int32, M * words(K), "out_signbits"),
            _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(grads.device):
        code = load().s3gd_debug_topk_sign(*args, _stream(grads), int(sample_rank))
    _check("s3gd_debug_topk_sign", code)


def s3gd_debug_step(x: torch.Tensor, grads: torch.Tensor, K: int, lr: float, ws: torch.Tensor, sample_rank: int,
                    opt_idx: Optional[torch.Tensor] = None, opt_signbits: Optional[torch.Tensor] = None,
                    opt_vote: Optional[torch.Tensor] = None, prevote_rank: int = 0) -> None:
    """s3gd_step with the sampling ranks of the two filter thresholds forced (0: the library's own)."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (_ptr(x, torch.float32, d, "x"), g, M, d, K, ctypes.c_float(lr),
            _ptr(opt_idx, torch.int32, M * K, "opt_idx"), _ptr(opt_signbits, torch.int32, M * words(K), "opt_signbits"),
            _ptr(opt_vote, torch.int8, d, "opt_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(x.device):
        code = load().s3gd_debug_step(*args, _stream(x), int(sample_rank), int(prevote_rank))
    _check("s3gd_debug_step", code)


def s3gd_vote_apply(x: torch.Tensor, msg: torch.Tensor, n_groups: int, group_stride: int, M_group: int, K: int,
                    lr: float, ws: torch.Tensor, opt_vote: Optional[torch.Tensor] = None) -> None:
    """Vote over a message gathered from n_groups senders (each piece: indices then sign words) fused with the update."""
    d = x.numel()
    need = (n_groups - 1) * group_stride + M_group * (K + words(K)) if n_groups > 0 else 0
    args = (_ptr(x, torch.float32, name="x"), _ptr(msg, torch.int32, need, "msg"), n_groups, group_stride, M_group, K, d,
            ctypes.c_float(lr), _ptr(opt_vote, torch.int8, d, "opt_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(x.device):
        code = load().s3gd_vote_apply(*args, _stream(x))
    _check("s3gd_vote_apply", code)


def s3gd_vote_counts(idx: torch.Tensor, signbits: torch.Tensor, M: int, K: int, d: int, out_counts: torch.Tensor,
                     opt_bad_count: Optional[torch.Tensor] = None) -> None:
    """Vote sums of M workers into out_counts: uint8 [d_padded] (128 + sum) or int32 [d_padded] (sum)."""
    if out_counts.dtype == torch.uint8:
        per, p = 1, _ptr(out_counts, torch.uint8, d, "out_counts")
    else:
        per, p = 4, _ptr(out_counts, torch.int32, d, "out_counts")
    args = (_ptr(idx, torch.int32, M * K, "idx"), _ptr(signbits, torch.int32, M * words(K), "signbits"), M, K, d,
            out_counts.numel(), p, per, _ptr(opt_bad_count, torch.int32, 1, "opt_bad_count"))
    with torch.cuda.device(out_counts.device):
        code = load().s3gd_vote_counts(*args, _stream(out_counts))
    _check("s3gd_vote_counts", code)


def s3gd_encode_vote2(src: torch.Tensor, out_words: torch.Tensor, n_summed: int = 1) -> None:
    """Two-bit form of the vote from int32 sums, from summed biased bytes (uint8) or from an int8 vote."""
    n = src.numel()
    if src.dtype == torch.int32:
        kind, p = 0, _ptr(src, torch.int32, name="src")
    elif src.dtype == torch.uint8:
        kind, p = 1, _ptr(src, torch.uint8, name="src")
    else:
        kind, p = 2, _ptr(src, torch.int8, name="src")
    args = (p, kind, n_summed, n, _ptr(out_words, torch.int32, (n + 15) // 16, "out_words"))
    with torch.cuda.device(src.device):
        code = load().s3gd_encode_vote2(*args, _stream(src))
    _check("s3gd_encode_vote2", code)


def s3gd_apply_vote2(x: torch.Tensor, words2: torch.Tensor, lr: float, opt_vote: Optional[torch.Tensor] = None) -> None:
    """x <- x - lr * vote with the vote in its two-bit form."""
    d = x.numel()
    args = (_ptr(x, torch.float32, name="x"), _ptr(words2, torch.int32, (d + 15) // 16, "words"), d, ctypes.c_float(lr),
            _ptr(opt_vote, torch.int8, d, "opt_vote"))
    with torch.cuda.device(x.device):
        code = load().s3gd_apply_vote2(*args, _stream(x))
    _check("s3gd_apply_vote2", code)


def sparse_piece_words(cap: int) -> int:
    """uint32 words of one sparse message: its count, cap indices, ceil(cap / 32) sign words."""
    return 1 + int(cap) + words(cap)


def s3gd_sparse_workspace_bytes(n: int) -> int:
    return int(load().s3gd_sparse_workspace_bytes(int(n)))


def s3gd_encode_vote_sparse(src: torch.Tensor, out_piece: torch.Tensor, cap: int, ws: torch.Tensor,
                            index_base: int = 0, n_summed: int = 1) -> None:
    """Sparse form (count, ascending indices, sign words) of the votes in src: int32 sums, summed biased bytes or int8."""
    n = src.numel()
    if src.dtype == torch.int32:
        kind, p = 0, _ptr(src, torch.int32, name="src")
    elif src.dtype == torch.uint8:
        kind, p = 1, _ptr(src, torch.uint8, name="src")
    else:
        kind, p = 2, _ptr(src, torch.int8, name="src")
    args = (p, kind, n_summed, n, index_base, cap, _ptr(out_piece, torch.int32, sparse_piece_words(cap), "out_piece"),
            _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(src.device):
        code = load().s3gd_encode_vote_sparse(*args, _stream(src))
    _check("s3gd_encode_vote_sparse", code)


def s3gd_apply_vote_sparse(x: torch.Tensor, pieces: torch.Tensor, n_pieces: int, piece_stride: int, cap: int, lr: float,
                           opt_bad_count: Optional[torch.Tensor] = None) -> None:
    """x <- x - lr * vote from n_pieces sparse messages lying piece_stride words apart."""
    d = x.numel()
    need = (n_pieces - 1) * piece_stride + sparse_piece_words(cap)
    args = (_ptr(x, torch.float32, name="x"), _ptr(pieces, torch.int32, need, "pieces"), n_pieces, piece_stride, cap, d,
            ctypes.c_float(lr), _ptr(opt_bad_count, torch.int32, 1, "opt_bad_count"))
    with torch.cuda.device(x.device):
        code = load().s3gd_apply_vote_sparse(*args, _stream(x))
    _check("s3gd_apply_vote_sparse", code)


PHASES = ("sample", "filter", "threshold", "emit", "apply")


def s3gd_profile_begin(max_steps: int) -> None:
    _check("s3gd_profile_begin", load().s3gd_profile_begin(int(max_steps)))


def s3gd_profile_begin_filter(max_steps: int) -> None:
    """As s3gd_profile_begin, but only the filter pass is bracketed by events (the other phases read 0)."""
    _check("s3gd_profile_begin_filter", load().s3gd_profile_begin_filter(int(max_steps)))


def s3gd_profile_begin_filter_every(max_steps: int, every: int) -> None:
    """As s3gd_profile_begin_filter with only every `every`-th step recorded (at most max_steps of them)."""
    _check("s3gd_profile_begin_filter_every", load().s3gd_profile_begin_filter_every(int(max_steps), int(every)))


def s3gd_profile_end(max_steps: int):
    """Returns (per-step list of 5 phase durations in ms, kernels enqueued since s3gd_profile_begin)."""
    buf = (ctypes.c_float * (5 * max_steps))()
    n = ctypes.c_int(0)
    launches = ctypes.c_uint64(0)
    _check("s3gd_profile_end", load().s3gd_profile_end(buf, ctypes.byref(n), ctypes.byref(launches)))
    steps = [[buf[5 * i + k] for k in range(5)] for i in range(n.value)]
    return steps, int(launches.value)


def s3gd_noalloc_max_d() -> int:
    return int(load().s3gd_noalloc_max_d())


def s3gd_majority_vote_noalloc(idx: torch.Tensor, signbits: torch.Tensor, M: int, K: int, d: int,
                               out_vote: torch.Tensor, opt_bad_count: Optional[torch.Tensor] = None) -> None:
    """Majority vote whose counters live inside the library: no workspace argument, nothing allocated.

    For callers that cannot obtain device memory where they vote (see include/s3gd.h).  d must not
    exceed s3gd_noalloc_max_d(); calls on one device share the built-in counters, so do not overlap them.
    """
    args = (_ptr(idx, torch.int32, M * K, "idx"), _ptr(signbits, torch.int32, M * words(K), "signbits"), M, K, d,
            _ptr(out_vote, torch.int8, d, "out_vote"), _ptr(opt_bad_count, torch.int32, 1, "opt_bad_count"))
    with torch.cuda.device(out_vote.device):
        code = load().s3gd_majority_vote_noalloc(*args, _stream(out_vote))
    _check("s3gd_majority_vote_noalloc", code)


def s3gd_step_ex(x: torch.Tensor, grads: torch.Tensor, K: int, lr: float, ws: torch.Tensor,
                 err: Optional[torch.Tensor] = None, eta: float = 1.0,
                 v: Optional[torch.Tensor] = None, mu: float = 0.0,
                 opt_idx: Optional[torch.Tensor] = None, opt_signbits: Optional[torch.Tensor] = None,
                 opt_vote: Optional[torch.Tensor] = None) -> None:
    """The fused step with optional error memory err [M, d] (updated in place) and momentum v [d]."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (_ptr(x, torch.float32, d, "x"), g, _ptr(err, torch.float32, M * d, "err"), ctypes.c_float(eta),
            _ptr(v, torch.float32, d, "v"), ctypes.c_float(mu), M, d, K, ctypes.c_float(lr),
            _ptr(opt_idx, torch.int32, M * K, "opt_idx"), _ptr(opt_signbits, torch.int32, M * words(K), "opt_signbits"),
            _ptr(opt_vote, torch.int8, d, "opt_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(x.device):
        code = load().s3gd_step_ex(*args, _stream(x))
    _check("s3gd_step_ex", code)


def s3gd_apply_momentum(x: torch.Tensor, v: torch.Tensor, vote: torch.Tensor, mu: float, lr: float) -> None:
    """v <- mu * v + vote; x <- x - lr * v, in place."""
    d = x.numel()
    args = (_ptr(x, torch.float32, name="x"), _ptr(v, torch.float32, d, "v"), _ptr(vote, torch.int8, d, "vote"), d,
            ctypes.c_float(mu), ctypes.c_float(lr))
    with torch.cuda.device(x.device):
        code = load().s3gd_apply_momentum(*args, _stream(x))
    _check("s3gd_apply_momentum", code)


def s3gd_randk_sign(grads: torch.Tensor, K: int, seed: int, step: int, out_idx: torch.Tensor,
                    out_signbits: torch.Tensor, ws: torch.Tensor) -> None:
    """RandKSign: out_idx [M, K] = pi(0..K-1) per worker (generation order), out_signbits [M, ceil(K/32)]."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (g, M, d, K, seed & 0xFFFFFFFF, step & 0xFFFFFFFF, _ptr(out_idx, torch.int32, M * K, "out_idx"),
            _ptr(out_signbits, torch.int32, M * words(K), "out_signbits"),
            _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(grads.device):
        code = load().s3gd_randk_sign(*args, _stream(grads))
    _check("s3gd_randk_sign", code)


def s3gd_step_randk(x: torch.Tensor, grads: torch.Tensor, K: int, lr: float, seed: int, step: int, ws: torch.Tensor,
                    opt_idx: Optional[torch.Tensor] = None, opt_signbits: Optional[torch.Tensor] = None,
                    opt_vote: Optional[torch.Tensor] = None) -> None:
    """The fused step with RandKSign in place of TopKSign."""
    g = _ptr(grads, torch.float32, name="grads")
    M, d = grads.shape
    args = (_ptr(x, torch.float32, d, "x"), g, M, d, K, ctypes.c_float(lr), seed & 0xFFFFFFFF, step & 0xFFFFFFFF,
            _ptr(opt_idx, torch.int32, M * K, "opt_idx"), _ptr(opt_signbits, torch.int32, M * words(K), "opt_signbits"),
            _ptr(opt_vote, torch.int8, d, "opt_vote"), _ptr(ws, torch.uint8, name="ws"), ws.numel())
    with torch.cuda.device(x.device):
        code = load().s3gd_step_randk(*args, _stream(x))
    _check("s3gd_step_randk", code)
