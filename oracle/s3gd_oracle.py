"""CPU oracle for one S3GD-MV compression / aggregation / update step.

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct
statement of what the hot path computes.  It shares no code with the CUDA
library and must never be imported by it; only the tests, the smoke check and
the benchmark's CPU-baseline leg may call it.

What is computed (paper: Park & Lee, "Sparse-SignSGD with Majority Vote"):

* TopK / TopKSign (Section 2.1, Eq. (3) ``TopK`` and Eq. (4) ``TopKSign``):
  keep the K entries of largest magnitude, replace them by their sign.
* Majority vote (Section 2.2, "Majority vote" paragraph and Algorithm 1):
  sgn of the sum over workers of the ternary vectors; coordinates nobody voted
  on, and exact ties, stay 0 because sgn(0) = 0 in the paper's definition.
* Model update (Section 2.2, Eq. (7)): x <- x - delta * vote.

Readings where the paper is silent (all listed in the design notes):

* magnitude order is the unsigned order of the fp32 bit pattern with the sign
  bit cleared (so denormals, Inf and NaN need no special case);
* exactly K entries are kept; among equal magnitudes the lower index wins;
* a selected entry votes with its IEEE sign bit (+0 votes +1, -0 votes -1), so
  that every worker has exactly K non-zero votes as Section 2.2 states;
* the K indices are listed ascending, 0-based; sign bit j belongs to index j,
  packed LSB-first into 32-bit words (1 = negative), padding bits 0;
* the update is one fp32 round-to-nearest operation: x - lr or x + lr.

All integer results are exact, so GPU output must equal them bit for bit.
Also here: error compensation (Eq. (5)-(6)), the momentum update (Section 4.7), the
random-K variant (Section 3.4, Algorithm 2), and the server's message to the workers
(Section 2.2, "Majority vote": the voted ternary vector, zero outside the union of the
workers' supports) in two transmitted forms with the paper's bit counts beside them.

Parity status: every function below is pinned by tests that do not call it to
build their expectation (brute-force rank counting, the printed worked
example, the K = N and M = 1 special cases of Section 3.3, invariants).
"""
from __future__ import annotations

import numpy as np

ABS_MASK = np.uint32(0x7FFFFFFF)


def _as_bits(grads: np.ndarray) -> np.ndarray:
    g = np.ascontiguousarray(grads, dtype=np.float32)
    if g.ndim != 2:
        raise ValueError("grads must be [M, d]")
    return g.view(np.uint32)


def magnitude_keys(row_bits: np.ndarray) -> np.ndarray:
    """|u| as an ordered unsigned integer: the bit pattern without its sign bit."""
    return row_bits & ABS_MASK


def pack_sign_bits(neg: np.ndarray) -> np.ndarray:
    """Pack booleans (True = negative) LSB-first into uint32 words, zero padded."""
    K = int(neg.shape[0])
    words = np.zeros((K + 31) // 32, dtype=np.uint32)
    for j in range(K):
        if neg[j]:
            words[j >> 5] |= np.uint32(1) << np.uint32(j & 31)
    return words


def _pack_sign_bits_fast(neg: np.ndarray) -> np.ndarray:
    """Same packing with numpy bit ops (checked against pack_sign_bits in the tests)."""
    K = int(neg.shape[0])
    W = (K + 31) // 32
    padded = np.zeros(W * 32, dtype=np.uint8)
    padded[:K] = neg
    by = np.packbits(padded.reshape(W, 32), axis=1, bitorder="little")  # [W, 4] bytes
    return by.view("<u4").reshape(W).astype(np.uint32)


def topk_sign(grads: np.ndarray, K: int):
    """TopKSign of every worker's gradient, Eq. (3)-(4), in transmitted form.

    Returns (idx [M, K] uint32 ascending, signbits [M, ceil(K/32)] uint32).
    Definition written out: order all coordinates by (magnitude descending,
    index ascending), keep the first K, list them by ascending index.
    """
    bits = _as_bits(grads)
    M, d = bits.shape
    if not 0 <= K <= d:
        raise ValueError("K must be in [0, d]")
    idx = np.zeros((M, K), dtype=np.uint32)
    sgn = np.zeros((M, (K + 31) // 32), dtype=np.uint32)
    for m in range(M):
        key = magnitude_keys(bits[m]).astype(np.int64)
        # a stable sort of the negated key puts equal magnitudes in index order
        order = np.argsort(-key, kind="stable")
        chosen = np.sort(order[:K])
        idx[m] = chosen.astype(np.uint32)
        sgn[m] = _pack_sign_bits_fast((bits[m][chosen] >> np.uint32(31)).astype(bool))
    return idx, sgn


def majority_vote(idx: np.ndarray, signbits: np.ndarray, M: int, K: int, d: int):
    """sgn of the summed votes, Algorithm 1 / "Majority vote" paragraph.

    Returns (vote [d] int8 in {-1, 0, +1}, n_out_of_range).  Repeated indices
    add up; an index >= d is skipped and counted.
    """
    idx = np.asarray(idx, dtype=np.uint32).reshape(M, K)
    signbits = np.asarray(signbits, dtype=np.uint32).reshape(M, (K + 31) // 32)
    count = np.zeros(d, dtype=np.int64)
    bad = 0
    j = np.arange(K)
    for m in range(M):
        neg = (signbits[m][j >> 5] >> (j & 31).astype(np.uint32)) & np.uint32(1)
        s = 1 - 2 * neg.astype(np.int64)
        ok = idx[m] < d
        bad += int(K - ok.sum())
        np.add.at(count, idx[m][ok].astype(np.int64), s[ok])
    vote = (count > 0).astype(np.int8) - (count < 0).astype(np.int8)
    return vote, bad


def apply_vote(x: np.ndarray, vote: np.ndarray, lr) -> np.ndarray:
    """x <- x - lr * vote, Eq. (7), in fp32 with one rounding; vote 0 leaves x's bits alone."""
    x = np.asarray(x, dtype=np.float32)
    lr32 = np.float32(lr)
    out = x.copy()
    pos = vote > 0
    neg = vote < 0
    out[pos] = (x[pos] - lr32).astype(np.float32)
    out[neg] = (x[neg] + lr32).astype(np.float32)
    return out


def step(x: np.ndarray, grads: np.ndarray, K: int, lr):
    """One whole step of Algorithm 1 without error memory: send, vote, update.

    Returns (x_new, idx, signbits, vote).
    """
    M, d = grads.shape
    idx, sgn = topk_sign(grads, K)
    vote, _ = majority_vote(idx, sgn, M, K, d)
    return apply_vote(x, vote, lr), idx, sgn, vote


# --------------------------------------------------------------------------
# The lines of Algorithm 1 around the step: error compensation before it
# (Section 2.2, Eq. (5)-(6)) and the momentum form of the update after it
# (Section 4.7, the two displays that replace Eq. (7)).
# --------------------------------------------------------------------------

def error_feedback_step(x, grads_tilde, err, eta, K: int, lr, topk=None):
    """Algorithm 1 with error memory, one iteration for all workers.

    g_m = g~_m + eta * e_m            (Eq. (5); fp32: one rounding for the product, one for the sum)
    e_m <- g_m - TopK(g_m)            (Eq. (6): g_m with its K kept entries set to zero)
    x   <- x - lr * sgn(sum_m TopKSign(g_m))

    Returns (x_new, err_new, idx, signbits, vote).  TopK(g) keeps the values of the K
    selected entries, so err_new equals g off the support and is exactly +0 on it.
    """
    gt = np.asarray(grads_tilde, dtype=np.float32)
    e = np.asarray(err, dtype=np.float32)
    M, d = gt.shape
    eta32 = np.float32(eta)
    g = (gt + (eta32 * e).astype(np.float32)).astype(np.float32)
    idx, sgn = (topk or topk_sign)(g, K)
    vote, _ = majority_vote(idx, sgn, M, K, d)
    err_new = g.copy()
    for m in range(M):
        err_new[m][idx[m].astype(np.int64)] = np.float32(0.0)
    return apply_vote(x, vote, lr), err_new, idx, sgn, vote


def apply_vote_momentum(x, v, vote, mu, lr):
    """Momentum form of the update (Section 4.7): v <- mu * v + vote ; x <- x - lr * v.

    fp32 with one rounding per operation: fl(mu*v), fl(. + vote), fl(lr*v), fl(x - .).
    Returns (x_new, v_new).
    """
    x = np.asarray(x, dtype=np.float32)
    v = np.asarray(v, dtype=np.float32)
    mu32, lr32 = np.float32(mu), np.float32(lr)
    v_new = ((mu32 * v).astype(np.float32) + np.asarray(vote).astype(np.float32)).astype(np.float32)
    x_new = (x - (lr32 * v_new).astype(np.float32)).astype(np.float32)
    return x_new, v_new


# --------------------------------------------------------------------------
# Random-K variant (Section 3.4, Algorithm 2): RandKSign keeps K coordinates chosen
# uniformly at random instead of the K largest.  The paper names no generator; the
# reading taken here: worker m at iteration t keeps the coordinates
# pi(0), pi(1), ..., pi(K-1) of a keyed pseudo-random permutation pi of [0, d), in
# that order (a K-subset without repetition; with the key shared, the indices
# themselves would not even have to be transmitted).  pi is a 4-round balanced
# Feistel network on 2h bits (2^(2h) >= d) with cycle walking into [0, d)
# (Black & Rogaway, "Ciphers with arbitrary finite domains", 2002); its round
# function is the 32-bit integer mixer "lowbias32" (C. Wellons, 2018):
#   v ^= v >> 16; v *= 0x7feb352d; v ^= v >> 15; v *= 0x846ca68b; v ^= v >> 16.
# Each side (this file, the CUDA kernels) implements these definitions on its own.
# --------------------------------------------------------------------------

def _lowbias32(v: np.ndarray) -> np.ndarray:
    v = v.astype(np.uint64)
    v ^= v >> np.uint64(16)
    v = (v * np.uint64(0x7FEB352D)) & np.uint64(0xFFFFFFFF)
    v ^= v >> np.uint64(15)
    v = (v * np.uint64(0x846CA68B)) & np.uint64(0xFFFFFFFF)
    v ^= v >> np.uint64(16)
    return v


def randk_round_keys(seed: int, worker: int, step: int) -> np.ndarray:
    """Four 32-bit round keys of worker `worker` at iteration `step` under `seed`."""
    keys = np.zeros(4, dtype=np.uint64)
    base = (int(seed) & 0xFFFFFFFF) ^ ((int(worker) * 0x9E3779B9) & 0xFFFFFFFF) ^ ((int(step) * 0x85EBCA6B) & 0xFFFFFFFF)
    for r in range(4):
        keys[r] = _lowbias32(np.array([(base + (r + 1) * 0x9E3779B9) & 0xFFFFFFFF], dtype=np.uint64))[0]
    return keys


def randk_permutation(j: np.ndarray, d: int, keys: np.ndarray) -> np.ndarray:
    """pi(j) for every entry of j (all < d): Feistel on 2h bits, walked until the value is below d."""
    h = 1
    while (1 << (2 * h)) < d:
        h += 1
    mask = np.uint64((1 << h) - 1)
    v = np.asarray(j, dtype=np.uint64).copy()
    todo = np.ones(v.shape, dtype=bool)
    while todo.any():
        left, right = v[todo] >> np.uint64(h), v[todo] & mask
        for r in range(4):
            f = _lowbias32(right ^ keys[r]) & mask
            left, right = right, left ^ f
        v[todo] = (left << np.uint64(h)) | right
        todo &= v >= np.uint64(d)                  # cycle walking: outside [0, d) -> apply pi again
    return v.astype(np.uint32)


def randk_sign(grads: np.ndarray, K: int, seed: int, step: int):
    """RandKSign of every worker (Algorithm 2, the "send" line) in transmitted form.

    Returns (idx [M, K] uint32 in generation order pi(0..K-1), signbits [M, ceil(K/32)]);
    sign bit j is the IEEE sign of the entry at idx[j].
    """
    bits = _as_bits(grads)
    M, d = bits.shape
    if not 0 <= K <= d:
        raise ValueError("K must be in [0, d]")
    idx = np.zeros((M, K), dtype=np.uint32)
    sgn = np.zeros((M, (K + 31) // 32), dtype=np.uint32)
    for m in range(M):
        idx[m] = randk_permutation(np.arange(K, dtype=np.uint64), d, randk_round_keys(seed, m, step))
        sgn[m] = _pack_sign_bits_fast((bits[m][idx[m].astype(np.int64)] >> np.uint32(31)).astype(bool))
    return idx, sgn


def randk_step(x: np.ndarray, grads: np.ndarray, K: int, lr, seed: int, step: int):
    """One iteration of Algorithm 2: RandKSign, majority vote, update.  Returns (x_new, idx, signbits, vote)."""
    M, d = grads.shape
    idx, sgn = randk_sign(grads, K, seed, step)
    vote, _ = majority_vote(idx, sgn, M, K, d)
    return apply_vote(x, vote, lr), idx, sgn, vote


# --------------------------------------------------------------------------
# The server's side of the exchange (Section 2.2, "Majority vote", and Algorithm 1's
# "send"/"receive" lines): vote counts as sums, and the voted vector in the two forms
# in which it can travel back to the workers.
# --------------------------------------------------------------------------

def vote_counts(idx: np.ndarray, signbits: np.ndarray, M: int, K: int, d: int) -> np.ndarray:
    """count[n] = sum over workers of their vote on coordinate n (+1, -1 or nothing), as int64.

    majority_vote() is the sign of this.  Sums of several groups of workers add up to the
    sum of all of them, which is what lets a server be split over coordinate ranges."""
    idx = np.asarray(idx, dtype=np.uint32).reshape(M, K)
    signbits = np.asarray(signbits, dtype=np.uint32).reshape(M, (K + 31) // 32)
    count = np.zeros(d, dtype=np.int64)
    for m in range(M):
        for j in range(K):
            n = int(idx[m, j])
            if n < d:
                neg = (int(signbits[m, j >> 5]) >> (j & 31)) & 1
                count[n] += -1 if neg else 1
    return count


def encode_vote_2bit(vote: np.ndarray) -> np.ndarray:
    """Dense form: two bits per coordinate, 16 coordinates per uint32 word, LSB first.

    Bit 0 of a pair says "moved", bit 1 says "negative": 0 -> 00, +1 -> 01, -1 -> 11.
    Padding pairs of the last word are 00."""
    v = np.asarray(vote, dtype=np.int8)
    d = v.shape[0]
    words = np.zeros((d + 15) // 16, dtype=np.uint32)
    for n in range(d):
        code = 0 if v[n] == 0 else (1 if v[n] > 0 else 3)
        words[n >> 4] |= np.uint32(code << (2 * (n & 15)))
    return words


def decode_vote_2bit(words: np.ndarray, d: int) -> np.ndarray:
    """Inverse of encode_vote_2bit (the pair 10 never occurs; it decodes as 0)."""
    w = np.asarray(words, dtype=np.uint32)
    vote = np.zeros(d, dtype=np.int8)
    for n in range(d):
        code = (int(w[n >> 4]) >> (2 * (n & 15))) & 3
        vote[n] = 1 if code == 1 else (-1 if code == 3 else 0)
    return vote


def encode_vote_sparse(vote: np.ndarray):
    """Sparse form: the non-zero coordinates, ascending, and their sign bits -- the same
    layout as a worker's message (uint32 indices; bit j of the sign words belongs to
    index j, LSB first, 1 = negative, zero padding).  Returns (idx [n], signbits [ceil(n/32)])."""
    v = np.asarray(vote, dtype=np.int8)
    where = [n for n in range(v.shape[0]) if v[n] != 0]
    idx = np.array(where, dtype=np.uint32)
    return idx, pack_sign_bits(np.array([v[n] < 0 for n in where], dtype=bool))


def decode_vote_sparse(idx: np.ndarray, signbits: np.ndarray, d: int) -> np.ndarray:
    """Inverse of encode_vote_sparse.  An index >= d is ignored."""
    vote = np.zeros(d, dtype=np.int8)
    idx = np.asarray(idx, dtype=np.uint32)
    sb = np.asarray(signbits, dtype=np.uint32)
    for j in range(idx.shape[0]):
        n = int(idx[j])
        if n < d:
            vote[n] = -1 if (int(sb[j >> 5]) >> (j & 31)) & 1 else 1
    return vote


def uplink_bits(K: int, N: int) -> float:
    """Bits one worker sends per round as Section 2.2 counts them: K + K log2(N / K)."""
    return 0.0 if K == 0 else K + K * float(np.log2(N / K))


def downlink_bits(n_voted: int, N: int) -> float:
    """Bits the server sends per round as Section 2.2 counts them: |N^t| + |N^t| log2(N / |N^t|)."""
    return uplink_bits(n_voted, N)


# --------------------------------------------------------------------------
# A second, faster route to the same selected set (threshold + tie fill), and
# an O(d) certificate check.  Both are pinned against topk_sign() in the tests;
# they exist so that rows of 1e7..1e9 elements can be checked in seconds.
# --------------------------------------------------------------------------

def topk_sign_threshold(grads: np.ndarray, K: int):
    """Same output as topk_sign(), via the threshold form of Eq. (3).

    rho = K-th largest magnitude (np.partition); everything above rho is kept,
    and the remaining places go to the lowest indices whose magnitude equals rho.
    """
    bits = _as_bits(grads)
    M, d = bits.shape
    if not 0 <= K <= d:
        raise ValueError("K must be in [0, d]")
    idx = np.zeros((M, K), dtype=np.uint32)
    sgn = np.zeros((M, (K + 31) // 32), dtype=np.uint32)
    if K == 0:
        return idx, sgn
    for m in range(M):
        key = magnitude_keys(bits[m])
        rho = np.partition(key, d - K)[d - K]
        above = np.flatnonzero(key > rho)
        ties = np.flatnonzero(key == rho)[: K - above.shape[0]]
        chosen = np.sort(np.concatenate([above, ties]))
        idx[m] = chosen.astype(np.uint32)
        sgn[m] = _pack_sign_bits_fast((bits[m][chosen] >> np.uint32(31)).astype(bool))
    return idx, sgn


def check_topk_sign_row(row: np.ndarray, K: int, idx: np.ndarray, signbits: np.ndarray) -> str:
    """Decide in O(d) whether (idx, signbits) is THE TopKSign message of ``row``.

    The answer is unique under the lowest-index tie rule, so a set that passes
    equals topk_sign()'s.  Returns "" when correct, else a description of the
    first violated condition:
      1. K strictly ascending indices below d;
      2. with rho = smallest selected magnitude: no unselected magnitude > rho;
      3. every unselected entry of magnitude rho lies after the last selected
         entry of magnitude rho;
      4. sign bit j is the IEEE sign of row[idx[j]], padding bits are 0.
    """
    rb = np.ascontiguousarray(row, dtype=np.float32).view(np.uint32)
    d = rb.shape[0]
    idx = np.asarray(idx, dtype=np.uint32)
    signbits = np.asarray(signbits, dtype=np.uint32)
    if idx.shape != (K,) or signbits.shape != ((K + 31) // 32,):
        return "wrong shapes"
    if K == 0:
        return ""
    i64 = idx.astype(np.int64)
    if i64[-1] >= d or np.any(np.diff(i64) <= 0):
        return "indices not strictly ascending in range"
    key = magnitude_keys(rb)
    sel = np.zeros(d, dtype=bool)
    sel[i64] = True
    rho = key[i64].min()
    if np.any(key[~sel] > rho):
        return "an unselected entry exceeds the smallest selected magnitude"
    unsel_ties = np.flatnonzero((key == rho) & ~sel)
    sel_ties = np.flatnonzero((key == rho) & sel)
    if unsel_ties.size and unsel_ties[0] < sel_ties[-1]:
        return "tie at the threshold not resolved toward the lower index"
    want = _pack_sign_bits_fast((rb[i64] >> np.uint32(31)).astype(bool))
    if not np.array_equal(want, signbits):
        return "sign bits do not match the IEEE signs of the selected entries"
    return ""
