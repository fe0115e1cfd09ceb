"""Pins the CPU oracle to things other than itself (no GPU, no CUDA library).

Every expectation here comes from the paper's printed values, from a closed
form, from brute force on tiny inputs, or from an invariant of the definition;
none is produced by calling the function under test.  The last test plants
plausible mistakes into the oracle and checks that the pins notice each one.
"""
import json
import os

import numpy as np
import pytest

from oracle import s3gd_oracle as O
from paper_2302_07475_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def f32_bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def unpack(signbits_row, K):
    j = np.arange(K)
    return ((signbits_row[j >> 5] >> (j & 31).astype(np.uint32)) & 1).astype(np.int64)


# ---------------------------------------------------------------- brute force
def brute_topk_sign(row, K):
    """Rank counting, O(d^2), no sort: n is kept iff fewer than K entries beat it.

    j beats n when |u_j| > |u_n|, or |u_j| == |u_n| and j < n (Eq. (3) plus the
    lowest-index tie rule).  Magnitudes are compared as Python floats via abs(),
    not via bit patterns, so this is a different route to the order.
    """
    d = len(row)
    vals = [float(v) for v in row]
    kept = []
    for n in range(d):
        rank = 0
        for j in range(d):
            if abs(vals[j]) > abs(vals[n]) or (abs(vals[j]) == abs(vals[n]) and j < n):
                rank += 1
        if rank < K:
            kept.append(n)
    neg = [np.signbit(row[n]) for n in kept]
    return kept, neg


def brute_vote(per_worker, d):
    count = [0] * d
    for kept, neg in per_worker:
        for n, s in zip(kept, neg):
            count[n] += -1 if s else 1
    return [(c > 0) - (c < 0) for c in count]


def pin_bruteforce(orc):
    rng = np.random.default_rng(1)
    for trial in range(30):
        d = int(rng.integers(1, 17))
        M = int(rng.integers(1, 5))
        # few distinct magnitudes => ties everywhere, both signs, exact zeros
        levels = np.array([0.0, 0.25, 0.25, 1.0, 1.5, 7.0], dtype=np.float32)
        g = levels[rng.integers(0, len(levels), (M, d))] * rng.choice([-1.0, 1.0], (M, d)).astype(np.float32)
        if trial % 3 == 0:
            g = rng.standard_normal((M, d)).astype(np.float32)
        for K in range(d + 1):
            idx, sgn = orc.topk_sign(g, K)
            per_worker = []
            for m in range(M):
                kept, neg = brute_topk_sign(g[m], K)
                per_worker.append((kept, neg))
                assert idx[m].tolist() == kept
                assert unpack(sgn[m], K).tolist() == [int(b) for b in neg]
                # padding bits of the last word are zero
                if K % 32:
                    assert int(sgn[m][-1]) >> (K % 32) == 0
            vote, bad = orc.majority_vote(idx, sgn, M, K, d)
            assert bad == 0
            assert vote.tolist() == brute_vote(per_worker, d)


def test_bruteforce_tiny():
    pin_bruteforce(O)


# ------------------------------------------------------ printed worked example
def pin_example1(orc):
    with open(os.path.join(GOLD, "example1_power_of_representative_democracy.json")) as f:
        ex = json.load(f)
    col = np.array(ex["values_at_coordinate_n"], dtype=np.float32)
    assert np.sign(col.astype(np.float64).mean()) == ex["sign_of_full_precision_mean"]
    # Three workers, d = 4.  Coordinate 2 holds the example's values.  The other
    # coordinates are filled so that with K = 1 worker 1 keeps coordinate 2
    # (3 is its largest, and the only one above the example's bar |g| > 1)
    # while workers 2 and 3 keep a different coordinate.
    g = np.array([[0.5, -0.2, col[0], 0.1],
                  [0.9, 0.1, col[1], -0.2],
                  [0.01, -0.8, col[2], 0.02]], dtype=np.float32)
    x = np.zeros(4, dtype=np.float32)
    # signSGD with majority vote = every entry votes (K = d)
    _, _, _, vote_all = orc.step(x, g, 4, 1.0)
    assert int(vote_all[2]) == ex["signsgd_majority_vote"]
    # sparsified vote: only the confident worker takes part at coordinate 2
    xs, idx, _, vote_1 = orc.step(x, g, 1, 1.0)
    assert idx[:, 0].tolist() == [2, 0, 1]
    assert int(vote_1[2]) == ex["thresholded_majority_vote"]
    assert xs[2] == np.float32(-1.0)      # x - delta * (+1)


def test_example1_printed_values():
    pin_example1(O)


# ----------------------------------------------- closed-form special cases
def pin_gamma_one_is_signsgd_mv(orc):
    """Section 3.3, gamma = 1: the step equals signSGD with majority vote."""
    rng = np.random.default_rng(2)
    M, d = 7, 300
    g = rng.standard_normal((M, d)).astype(np.float32)
    g[:, ::17] = 0.0
    g[::2, ::34] = -0.0
    x = rng.standard_normal(d).astype(np.float32)
    lr = np.float32(0.01)
    x_new, idx, sgn, vote = orc.step(x, g, d, lr)
    for n in range(d):
        total = 0
        for m in range(M):
            total += -1 if np.signbit(g[m, n]) else 1
        want = (total > 0) - (total < 0)
        assert vote[n] == want
        assert x_new[n] == np.float32(np.float64(x[n]) - np.float64(lr) * want)
    assert all(idx[m].tolist() == list(range(d)) for m in range(M))


def pin_single_worker(orc):
    """Section 3.3, M = 1: the vote is TopKSign(g) itself; exactly K coordinates move by lr."""
    rng = np.random.default_rng(3)
    d, K = 500, 37
    g = rng.standard_normal((1, d)).astype(np.float32)
    x = (np.round(rng.standard_normal(d) * 1024) / 1024).astype(np.float32)
    lr = np.float32(0.125)                      # x on a 2^-10 grid: x -/+ lr is exact
    x_new, idx, sgn, vote = orc.step(x, g, K, lr)
    mags = np.abs(g[0].astype(np.float64))
    kth = np.sort(mags)[::-1][K - 1]
    want = np.where(mags >= kth, np.sign(g[0]), 0).astype(np.int64)   # no ties in continuous data
    assert np.array_equal(vote.astype(np.int64), want)
    assert int(np.count_nonzero(vote)) == K
    moved = x_new != x
    assert np.array_equal(moved, vote != 0)
    assert np.array_equal((x_new - x)[moved], (-lr * vote[moved]).astype(np.float32))


def test_special_cases():
    pin_gamma_one_is_signsgd_mv(O)
    pin_single_worker(O)


# ------------------------------------------------------------ invariants
def pin_invariants(orc):
    rng = np.random.default_rng(4)
    M, d = 6, 2000
    g = rng.standard_normal((M, d)).astype(np.float32)
    g = (np.round(g * 8) / 8).astype(np.float32)        # plenty of ties
    x = rng.standard_normal(d).astype(np.float32)
    lr = np.float32(1e-3)
    prev = None
    for K in (0, 1, 31, 32, 33, 200, 1999, 2000):
        x_new, idx, sgn, vote = orc.step(x, g, K, lr)
        # exactly K distinct ascending in-range indices per worker (Section 2.2)
        for m in range(M):
            assert idx[m].shape == (K,)
            assert np.all(np.diff(idx[m].astype(np.int64)) > 0)
            assert K == 0 or idx[m][-1] < d
        # sum of all counts equals the signed number of votes
        total = sum(K - 2 * int(unpack(sgn[m], K).sum()) for m in range(M))
        cnt = np.zeros(d, dtype=np.int64)
        for m in range(M):
            np.add.at(cnt, idx[m].astype(np.int64), 1 - 2 * unpack(sgn[m], K))
        assert cnt.sum() == total
        assert np.count_nonzero(vote) <= min(d, M * K)
        # permuting the workers changes nothing at the server
        perm = rng.permutation(M)
        xp, _, _, vp = orc.step(x, g[perm], K, lr)
        assert np.array_equal(vp, vote) and np.array_equal(f32_bits(xp), f32_bits(x_new))
        # negating every gradient keeps the support, flips signs and the vote
        xn, idxn, sgnn, vn = orc.step(x, -g, K, lr)
        assert np.array_equal(idxn, idx) and np.array_equal(vn, -vote)
        for m in range(M):
            assert np.array_equal(unpack(sgnn[m], K), 1 - unpack(sgn[m], K))
        # scaling a row by a power of two is exact and changes nothing
        g2 = g.copy()
        g2[1] *= np.float32(4.0)
        _, idx2, sgn2, _ = orc.step(x, g2, K, lr)
        assert np.array_equal(idx2, idx) and np.array_equal(sgn2, sgn)
        # supports are nested in K
        if prev is not None:
            for m in range(M):
                assert set(prev[m].tolist()) <= set(idx[m].tolist())
        prev = idx
        # the update moves voted coordinates by one correctly rounded fp32 operation
        want = (x.astype(np.float64) - np.float64(lr) * vote).astype(np.float32)
        assert np.array_equal(f32_bits(x_new)[vote != 0], f32_bits(want)[vote != 0])
        assert np.array_equal(f32_bits(x_new)[vote == 0], f32_bits(x)[vote == 0])


def test_invariants():
    pin_invariants(O)


def pin_apply_bits(orc):
    """vote 0 must leave the bit pattern alone (NaN payloads, -0); vote +-1 is one rounding."""
    x = np.array([0.0, -0.0, 1.0, np.nan, np.inf, 1e-40, 16777216.0, 0.1], dtype=np.float32)
    xb = f32_bits(x).copy()
    xb[3] = 0x7FC12345
    x = xb.view(np.float32)
    vote0 = np.zeros(8, dtype=np.int8)
    assert np.array_equal(f32_bits(orc.apply_vote(x, vote0, 0.5)), xb)
    votep = np.ones(8, dtype=np.int8)
    lr = np.float32(0.3)
    got = orc.apply_vote(x, votep, lr)
    want = (x.astype(np.float64) - np.float64(lr)).astype(np.float32)
    ok = ~np.isnan(want)
    assert np.array_equal(f32_bits(got)[ok], f32_bits(want)[ok])
    got = orc.apply_vote(x, -votep, lr)
    want = (x.astype(np.float64) + np.float64(lr)).astype(np.float32)
    assert np.array_equal(f32_bits(got)[ok], f32_bits(want)[ok])


def test_apply_bits():
    pin_apply_bits(O)


def pin_vote_semantics(orc):
    """Repeated indices add up; out-of-range indices are skipped and counted; ties give 0."""
    d, M, K = 10, 2, 4
    idx = np.array([[1, 1, 3, 9], [1, 3, 4, 12]], dtype=np.uint32)
    sgn = np.array([[0b0110], [0b0001]], dtype=np.uint32)   # w0: +,-,-,+   w1: -,+,+,+
    vote, bad = orc.majority_vote(idx, sgn, M, K, d)
    # coord1: +1 -1 -1 = -1 ; coord3: -1 +1 = 0 ; coord4: +1 ; coord9: +1 ; 12 skipped
    want = [0, -1, 0, 0, 1, 0, 0, 0, 0, 1]
    assert vote.tolist() == want and bad == 1


def test_vote_semantics():
    pin_vote_semantics(O)


def pin_downlink_forms(orc):
    """The voted vector in its two transmitted forms (Section 2.2, "Majority vote"): literal words for a
    hand-worked vector, exhaustive round trips over every ternary vector of length 7, and vote sums that
    add up over groups of workers and restrict to coordinate ranges (what a sharded server relies on)."""
    # worked by hand: pairs (bit 0 = moved, bit 1 = negative), coordinate n at bits 2(n mod 16) of word n div 16
    v = np.zeros(17, dtype=np.int8)
    v[[1, 5, 16]] = 1
    v[[2, 4, 15]] = -1
    #  n=1: 01<<2 = 0x4   n=2: 11<<4 = 0x30   n=4: 11<<8 = 0x300   n=5: 01<<10 = 0x400   n=15: 11<<30 = 0xC0000000
    assert orc.encode_vote_2bit(v).tolist() == [0xC0000734, 0x1]
    idx, sb = orc.encode_vote_sparse(v)
    assert idx.tolist() == [1, 2, 4, 5, 15, 16] and sb.tolist() == [0b010110]     # entries 1, 2, 4 are negative
    assert orc.decode_vote_2bit(np.array([0xC0000734, 0x1], np.uint32), 17).tolist() == v.tolist()
    assert orc.decode_vote_sparse(np.array([1, 2, 4, 5, 15, 16], np.uint32), np.array([0b010110], np.uint32), 17).tolist() == v.tolist()
    assert orc.decode_vote_2bit(np.array([0b10], np.uint32), 1).tolist() == [0]     # the unused pair
    assert orc.decode_vote_sparse(np.array([3, 99], np.uint32), np.array([0b10], np.uint32), 5).tolist() == [0, 0, 0, 1, 0]
    for code in range(3 ** 7):                      # every ternary vector of length 7
        t = np.array([(code // 3 ** i) % 3 - 1 for i in range(7)], dtype=np.int8)
        assert orc.decode_vote_2bit(orc.encode_vote_2bit(t), 7).tolist() == t.tolist()
        i, sgn = orc.encode_vote_sparse(t)
        assert i.shape[0] == np.count_nonzero(t) and np.all(np.diff(i.astype(np.int64)) > 0)
        assert orc.decode_vote_sparse(i, sgn, 7).tolist() == t.tolist()
    rng = np.random.default_rng(12)
    d, M, K = 300, 6, 40
    g = rng.standard_normal((M, d)).astype(np.float32)
    g[:, ::7] = np.abs(g[:, 1::7][:, : g[:, ::7].shape[1]])
    idx, sgn = orc.topk_sign(g, K)
    count = orc.vote_counts(idx, sgn, M, K, d)
    brute = np.zeros(d, dtype=np.int64)             # by definition: sum over workers of the ternary vectors
    for m in range(M):
        tern = np.zeros(d, dtype=np.int64)
        tern[idx[m]] = np.where(np.signbit(g[m][idx[m]]), -1, 1)
        brute += tern
    assert np.array_equal(count, brute)
    vote, _ = orc.majority_vote(idx, sgn, M, K, d)
    assert np.array_equal(np.sign(count).astype(np.int8), vote)
    halves = orc.vote_counts(idx[:2], sgn[:2], 2, K, d) + orc.vote_counts(idx[2:], sgn[2:], M - 2, K, d)
    assert np.array_equal(halves, count)
    x = rng.standard_normal(d).astype(np.float32)
    via2 = orc.apply_vote(x, orc.decode_vote_2bit(orc.encode_vote_2bit(vote), d), 0.37)
    vias = orc.apply_vote(x, orc.decode_vote_sparse(*orc.encode_vote_sparse(vote), d), 0.37)
    want = orc.apply_vote(x, vote, 0.37)
    assert np.array_equal(f32_bits(via2), f32_bits(want)) and np.array_equal(f32_bits(vias), f32_bits(want))
    # the bit counts as Section 2.2 writes them: K + K log2(N / K), equal to N at K = N (signSGD's one bit each)
    assert orc.uplink_bits(2 ** 10, 2 ** 20) == 2 ** 10 * 11 and orc.uplink_bits(4096, 4096) == 4096
    assert orc.downlink_bits(2 ** 10, 2 ** 20) == 2 ** 10 * 11 and orc.uplink_bits(0, 100) == 0.0


def test_downlink_forms():
    pin_downlink_forms(O)


def test_special_values_order():
    """NaN > Inf > finite > denormal > 0 in the bit-pattern order; signs taken from the sign bit."""
    g = np.array([[1.0, -np.inf, 1e-42, np.nan, -0.0, 3e38, -1e-45, 0.0]], dtype=np.float32)
    idx, sgn = O.topk_sign(g, 8)
    ranks = []
    for K in range(1, 9):
        i, _ = O.topk_sign(g, K)
        ranks.append(set(i[0].tolist()))
    order = [next(iter(ranks[0]))] + [next(iter(ranks[k] - ranks[k - 1])) for k in range(1, 8)]
    assert order == [3, 1, 5, 0, 2, 6, 4, 7]
    assert unpack(sgn[0], 8).tolist() == [0, 1, 0, 0, 1, 0, 1, 0]


# ----------------------------------------------------- packing helper pinned
def test_pack_helpers_agree():
    rng = np.random.default_rng(5)
    for K in (0, 1, 31, 32, 33, 64, 1000):
        neg = rng.random(K) < 0.5
        slow = O.pack_sign_bits(neg)
        assert np.array_equal(slow, O._pack_sign_bits_fast(neg))
        # written out once more from the layout statement: word j//32, bit j%32
        for j in range(K):
            assert ((int(slow[j // 32]) >> (j % 32)) & 1) == int(neg[j])


# ---------------------------------- threshold route and certificate check
@pytest.mark.parametrize("kind", ["normal", "all_equal", "zeros", "few_levels", "one_hot", "special", "ramp"])
def test_threshold_route_equals_definition(kind):
    M, d = 3, 1537
    if kind == "normal":
        g = np.random.default_rng(6).standard_normal((M, d)).astype(np.float32)
    else:
        g = W.edge_case_grads(kind, M, d).numpy()
    for K in (0, 1, 2, 100, 768, 1536, 1537):
        a = O.topk_sign(g, K)
        b = O.topk_sign_threshold(g, K)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
        for m in range(M):
            assert O.check_topk_sign_row(g[m], K, a[0][m], a[1][m]) == ""


def test_threshold_route_on_workload_shapes():
    s = W.spec("resnet50_ties", d=200_003, M=2)
    g = W.make_grads(s, "cpu").numpy()
    for K in (20, 200, 2000, 20000):
        a = O.topk_sign(g, K)
        b = O.topk_sign_threshold(g, K)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_certificate_rejects_wrong_answers():
    g = W.edge_case_grads("few_levels", 1, 400)[0].numpy()
    K = 150
    idx, sgn = O.topk_sign(g[None, :], K)
    idx, sgn = idx[0], sgn[0]
    assert O.check_topk_sign_row(g, K, idx, sgn) == ""
    key = f32_bits(g) & 0x7FFFFFFF
    rho = key[idx].min()
    sel = set(idx.tolist())
    # (a) swap the last selected tie for a later unselected tie: same magnitudes, wrong tie rule
    later = [n for n in range(400) if key[n] == rho and n not in sel]
    ties_sel = [n for n in idx.tolist() if key[n] == rho]
    assert later and ties_sel
    bad = np.array(sorted((sel - {ties_sel[0]}) | {later[-1]}), dtype=np.uint32)
    sb = O._pack_sign_bits_fast((f32_bits(g)[bad] >> 31).astype(bool))
    assert "tie" in O.check_topk_sign_row(g, K, bad, sb)
    # (b) replace a large entry by a small one
    small = [n for n in range(400) if key[n] < rho]
    big = [n for n in idx.tolist() if key[n] > rho]
    bad = np.array(sorted((sel - {big[0]}) | {small[0]}), dtype=np.uint32)
    sb = O._pack_sign_bits_fast((f32_bits(g)[bad] >> 31).astype(bool))
    assert "exceeds" in O.check_topk_sign_row(g, K, bad, sb)
    # (c) one flipped sign bit, (d) a set padding bit, (e) unsorted, (f) duplicate
    s2 = sgn.copy(); s2[1] ^= np.uint32(4)
    assert "sign" in O.check_topk_sign_row(g, K, idx, s2)
    s3 = sgn.copy(); s3[-1] |= np.uint32(1 << 31)
    assert "sign" in O.check_topk_sign_row(g, K, idx, s3)
    i2 = idx.copy(); i2[[3, 4]] = i2[[4, 3]]
    assert "ascending" in O.check_topk_sign_row(g, K, i2, sgn)
    i3 = idx.copy(); i3[5] = i3[4]
    assert "ascending" in O.check_topk_sign_row(g, K, i3, sgn)


# ------------------------------------------------ statistical closed forms
def test_support_statistics_match_closed_forms():
    """Independent rows: voter counts ~ Binomial(M, K/N) (Lemma 3); empty fraction (1-K/N)^M (Example 2)."""
    with open(os.path.join(GOLD, "closed_forms.json")) as f:
        cases = {(c["N"], c["K"], c["M"]): c for c in json.load(f)["cases"]}
    s = W.SPECS["tiny"]
    c = cases[(s.d, s.Ks[0], s.M)]
    g = W.make_grads(s, "cpu").numpy()
    idx, _ = O.topk_sign(g, s.Ks[0])
    voters = np.zeros(s.d, dtype=np.int64)
    for m in range(s.M):
        voters[idx[m]] += 1
    frac_voted = np.count_nonzero(voters) / s.d
    # alpha = 0.04898; std of the estimate ~ sqrt(alpha/N) ~ 8.6e-4
    assert abs(frac_voted - c["alpha"]) < 5 * 8.6e-4
    assert abs((voters == 0).mean() - c["p_empty"]) < 5 * 8.6e-4
    hist = np.bincount(voters, minlength=s.M + 1) / s.d
    assert abs(hist[1] - c["voter_count_pmf"][1]) < 5e-3
    assert abs(hist[2] - c["voter_count_pmf"][2]) < 1e-3


# ------------------------------------ error compensation and momentum (Eq. (5)-(6), Section 4.7)
def pin_error_feedback(orc):
    """Small integer-valued inputs (every fp32 operation exact), checked by brute force in Python ints."""
    rng = np.random.default_rng(11)
    M, d, K, eta = 3, 12, 4, 2.0
    x = np.zeros(d, dtype=np.float32)
    e = np.zeros((M, d), dtype=np.float32)
    sent_total = np.zeros((M, d), dtype=np.int64)        # sum over steps of TopK(g) (values)
    grad_total = np.zeros((M, d), dtype=np.int64)        # sum over steps of eta^(steps since) ... only for eta = 1 below
    for t in range(4):
        gt = rng.integers(-9, 10, (M, d)).astype(np.float32)
        g_int = gt.astype(np.int64) + int(eta) * e.astype(np.int64)          # Eq. (5) in exact arithmetic
        x_new, e_new, idx, sgn, vote = orc.error_feedback_step(x, gt, e, eta, K, 1.0)
        per_worker = []
        for m in range(M):
            kept, neg = brute_topk_sign(g_int[m].astype(np.float64), K)
            per_worker.append((kept, neg))
            assert idx[m].tolist() == kept
            want_e = g_int[m].copy(); want_e[kept] = 0                        # Eq. (6): g - TopK(g)
            assert e_new[m].astype(np.int64).tolist() == want_e.tolist()
            assert np.all(f32_bits(e_new[m][kept]) == 0)                      # +0, not -0
        assert vote.tolist() == brute_vote(per_worker, d)
        assert np.array_equal(x_new, x - vote.astype(np.float32))
        x, e = x_new, e_new
    # eta = 0: no memory, the step is the plain step on g~ and e = g~ - TopK(g~)
    gt = rng.standard_normal((M, d)).astype(np.float32)
    junk = rng.standard_normal((M, d)).astype(np.float32)
    x0 = rng.standard_normal(d).astype(np.float32)
    xa, ea, ia, sa, va = orc.error_feedback_step(x0, gt, junk, 0.0, K, 0.1)
    kept_all = [brute_topk_sign(gt[m], K)[0] for m in range(M)]
    assert [ia[m].tolist() for m in range(M)] == kept_all
    for m in range(M):
        off = np.ones(d, bool); off[kept_all[m]] = False
        assert np.array_equal(f32_bits(ea[m][off]), f32_bits(gt[m][off])) and np.all(ea[m][~off] == 0)
    # eta = 1 over several steps: what was sent plus what is remembered is everything that came in
    e = np.zeros((M, d), dtype=np.float32)
    for t in range(5):
        gt = rng.integers(-20, 21, (M, d)).astype(np.float32)
        g = gt + e
        _, e_new, idx, _, _ = orc.error_feedback_step(x0, gt, e, 1.0, K, 0.1)
        for m in range(M):
            sent_total[m][idx[m]] += g[m][idx[m]].astype(np.int64)
        grad_total += gt.astype(np.int64)
        e = e_new
    assert np.array_equal(sent_total + e.astype(np.int64), grad_total)


def pin_momentum(orc):
    from fractions import Fraction
    d = 6
    vote = np.array([1, -1, 0, 1, 0, -1], dtype=np.int8)
    # mu = 0: v is the vote and x moves exactly as in Eq. (7)
    x = np.array([0.5, -0.25, 3.0, 1e-3, -7.0, 0.1], dtype=np.float32)
    xn, vn = orc.apply_vote_momentum(x, np.full(d, 9.0, np.float32), vote, 0.0, 0.125)
    assert vn.tolist() == vote.astype(np.float32).tolist()
    want = (x.astype(np.float64) - 0.125 * vote).astype(np.float32)
    assert np.array_equal(xn, want)
    # mu = 1/2, lr = 1/4, the same vote T times: every quantity is a short dyadic fraction, exact in fp32
    x = np.zeros(d, dtype=np.float32); v = np.zeros(d, dtype=np.float32)
    fx = [Fraction(0)] * d; fv = [Fraction(0)] * d
    for t in range(8):
        x, v = orc.apply_vote_momentum(x, v, vote, 0.5, 0.25)
        fv = [Fraction(1, 2) * a + int(s) for a, s in zip(fv, vote)]
        fx = [a - Fraction(1, 4) * b for a, b in zip(fx, fv)]
        assert [Fraction(float(a)) for a in v] == fv and [Fraction(float(a)) for a in x] == fx
    # rounding order: fl(mu*v) first, then + vote; fl(lr*v) first, then x - .
    x1, v1 = orc.apply_vote_momentum(np.array([1.0], np.float32), np.array([0.1], np.float32),
                                     np.array([1], np.int8), np.float32(0.3), np.float32(0.7))
    mv = np.float32(np.float32(0.3) * np.float32(0.1))
    vv = np.float32(mv + np.float32(1.0))
    assert v1[0] == vv and x1[0] == np.float32(np.float32(1.0) - np.float32(np.float32(0.7) * vv))


def test_error_feedback_and_momentum():
    pin_error_feedback(O)
    pin_momentum(O)



# ------------------------------------------------ random-K variant (Section 3.4, Algorithm 2)
def pin_randk_subset(orc):
    """RandK keeps K distinct coordinates below d; K = d keeps every coordinate exactly once;
    the sign bit j is the sign of the entry at the j-th kept index."""
    rng = np.random.default_rng(5)
    for d in (1, 2, 3, 5, 16, 17, 64, 100, 1000, 4097, 70_001):
        for K in sorted({0, 1, d // 3, d - 1, d} - {-1}):
            M = 3
            g = rng.standard_normal((M, d)).astype(np.float32)
            g[:, ::7] = np.float32(-0.0)
            idx, sgn = orc.randk_sign(g, K, seed=d * 31 + K, step=K)
            assert idx.shape == (M, K) and sgn.shape == (M, (K + 31) // 32)
            for m in range(M):
                row = idx[m].astype(np.int64).tolist()
                assert all(0 <= n < d for n in row)
                assert len(set(row)) == K                                  # without repetition
                if K == d:
                    assert sorted(row) == list(range(d))
                assert unpack(sgn[m], K).tolist() == [int(f32_bits(g[m][n:n + 1])[0] >> 31) for n in row]
                if K % 32:
                    assert int(sgn[m][-1]) >> (K % 32) == 0                # unused bits are 0
    # a prefix property the transmitted form relies on: the K kept coordinates are the first K of the K' > K ones
    g = rng.standard_normal((2, 5000)).astype(np.float32)
    i1, _ = orc.randk_sign(g, 100, seed=9, step=4)
    i2, _ = orc.randk_sign(g, 700, seed=9, step=4)
    assert np.array_equal(i1, i2[:, :100])


def pin_randk_k_equals_d_is_signsgd_mv(orc):
    """With K = d nothing is dropped: Algorithm 2 is signSGD with majority vote whatever the permutation."""
    rng = np.random.default_rng(6)
    M, d = 7, 333
    g = rng.standard_normal((M, d)).astype(np.float32)
    x = rng.standard_normal(d).astype(np.float32)
    xn, idx, sgn, vote = orc.randk_step(x, g, d, 0.25, seed=1, step=0)
    total = np.where(np.signbit(g), -1, 1).sum(axis=0)
    assert vote.tolist() == np.sign(total).astype(np.int8).tolist()
    assert np.array_equal(xn, (x.astype(np.float64) - 0.25 * np.sign(total)).astype(np.float32))


def pin_randk_uniform_and_independent(orc):
    """Uniform K-subsets drawn independently per worker and per iteration: every coordinate is kept with
    probability K/N, the number of workers keeping one coordinate is Binomial(M, K/N) (Lemma 3) and the
    fraction nobody keeps is (1 - K/N)^M (Example 2)."""
    with open(os.path.join(GOLD, "closed_forms.json")) as f:
        cases = {(c["N"], c["K"], c["M"]): c for c in json.load(f)["cases"]}
    # one big draw
    N, K, M = 200000, 2000, 16
    c = cases[(N, K, M)]
    g = np.ones((M, N), dtype=np.float32)
    idx, _ = orc.randk_sign(g, K, seed=77, step=3)
    voters = np.zeros(N, dtype=np.int64)
    for m in range(M):
        voters[idx[m].astype(np.int64)] += 1
    sd = np.sqrt(c["alpha"] * (1 - c["alpha"]) / N)
    assert abs((voters == 0).mean() - c["p_empty"]) < 5 * sd
    hist = np.bincount(voters, minlength=M + 1) / N
    for k in (1, 2, 3):
        p = c["voter_count_pmf"][k]
        assert abs(hist[k] - p) < 5 * np.sqrt(p * (1 - p) / N) + 1e-6
    # many iterations on a small model: per-coordinate inclusion frequency is K/N everywhere (chi-square)
    N, K, M = 4096, 256, 8
    c = cases[(N, K, M)]
    g = np.ones((M, N), dtype=np.float32)
    steps = 120
    kept = np.zeros(N, dtype=np.int64)
    empty = 0
    first = np.zeros(N, dtype=np.int64)
    for t in range(steps):
        idx, _ = orc.randk_sign(g, K, seed=123, step=t)
        voters = np.zeros(N, dtype=np.int64)
        for m in range(M):
            voters[idx[m].astype(np.int64)] += 1
            first[int(idx[m][0])] += 1
        kept += voters
        empty += int((voters == 0).sum())
    draws = steps * M
    expect = draws * K / N                                          # 60 per coordinate
    chi2 = float(((kept - expect) ** 2 / (expect * (1 - K / N))).sum())
    assert abs(chi2 - (N - 1)) < 6 * np.sqrt(2 * (N - 1)), chi2     # chi-square with N-1 degrees of freedom
    assert abs(empty / (steps * N) - c["p_empty"]) < 5 * np.sqrt(c["p_empty"] * (1 - c["p_empty"]) / (steps * N))
    assert first.max() <= 8                                         # pi(0) is spread out, not stuck on a few values
    # different workers, iterations and seeds give different subsets
    a, _ = orc.randk_sign(g[:2], K, seed=1, step=0)
    b, _ = orc.randk_sign(g[:2], K, seed=1, step=1)
    c2, _ = orc.randk_sign(g[:2], K, seed=2, step=0)
    sets = [set(a[0].tolist()), set(a[1].tolist()), set(b[0].tolist()), set(c2[0].tolist())]
    for i in range(4):
        for j in range(i + 1, 4):
            assert len(sets[i] & sets[j]) < 60                       # expected overlap K^2/N = 16


def test_randk_pins():
    pin_randk_subset(O)
    pin_randk_k_equals_d_is_signsgd_mv(O)
    pin_randk_uniform_and_independent(O)


def test_randk_mixer_known_answers():
    """The 32-bit mixer and the Feistel network restated in Python integers, for a handful of inputs.

    A restatement is a guard against a slip of the vectorised uint64 arithmetic (a lost mask, a wrong
    shift), not a pin: it repeats the construction the oracle chose.  Section 3.4 fixes only the
    distribution of the kept set (K distinct coordinates, uniform, independent across workers and
    iterations), so what pins randk_* is the set of statistical and structural tests around this one:
    distinctness, the permutation at K = d, inclusion frequencies, the Binomial voter counts of Lemma 3
    and the empty fraction of Example 2."""
    def mix(v):
        v ^= v >> 16; v = (v * 0x7FEB352D) & 0xFFFFFFFF
        v ^= v >> 15; v = (v * 0x846CA68B) & 0xFFFFFFFF
        return v ^ (v >> 16)
    vals = [0, 1, 0xFFFFFFFF, 0x12345678, 0x80000000]
    assert O._lowbias32(np.array(vals, dtype=np.uint64)).tolist() == [mix(v) for v in vals]
    assert mix(0) == 0 and mix(1) != 1
    seed, worker, step, d = 42, 3, 7, 1000
    base = (seed ^ (worker * 0x9E3779B9) ^ (step * 0x85EBCA6B)) & 0xFFFFFFFF
    keys = [mix((base + (r + 1) * 0x9E3779B9) & 0xFFFFFFFF) for r in range(4)]
    assert O.randk_round_keys(seed, worker, step).tolist() == keys
    h = 5                                                            # 2^10 >= 1000
    def perm(v):
        while True:
            L, R = v >> h, v & 31
            for r in range(4):
                L, R = R, L ^ (mix(R ^ keys[r]) & 31)
            v = (L << h) | R
            if v < d:
                return v
    js = list(range(0, 1000, 37))
    assert O.randk_permutation(np.array(js), d, np.array(keys, dtype=np.uint64)).tolist() == [perm(j) for j in js]


# ------------------------------------------- the pins notice planted mistakes
ALL_PINS = [pin_bruteforce, pin_example1, pin_gamma_one_is_signsgd_mv, pin_single_worker,
            pin_invariants, pin_apply_bits, pin_vote_semantics, pin_error_feedback, pin_momentum,
            pin_randk_subset, pin_randk_k_equals_d_is_signsgd_mv, pin_randk_uniform_and_independent,
            pin_downlink_forms]


def _mutants():
    real_topk, real_vote, real_apply = O.topk_sign, O.majority_vote, O.apply_vote
    real_counts, real_enc2, real_encs = O.vote_counts, O.encode_vote_2bit, O.encode_vote_sparse

    def higher_index_wins(g, K):            # wrong tie rule
        M, d = g.shape
        i, s = real_topk(g[:, ::-1], K)
        i = (d - 1 - i.astype(np.int64))[:, ::-1].astype(np.uint32)
        out = np.zeros_like(s)
        for m in range(M):
            out[m] = O._pack_sign_bits_fast(np.signbit(g[m][i[m]]))
        return i, out

    def signed_not_magnitude(g, K):          # top-K of the signed value instead of |.|
        i, _ = real_topk(np.where(g > 0, g, 0).astype(np.float32), K)
        out = np.zeros((g.shape[0], (K + 31) // 32), dtype=np.uint32)
        for m in range(g.shape[0]):
            out[m] = O._pack_sign_bits_fast(np.signbit(g[m][i[m]]))
        return i, out

    def smallest_k(g, K):                    # ascending instead of descending
        with np.errstate(divide="ignore"):
            return real_topk((1.0 / (np.abs(g) + 1e-3)).astype(np.float32) * np.where(np.signbit(g), -1, 1).astype(np.float32), K)

    def inverted_sign_bits(g, K):            # 1 = positive
        i, s = real_topk(g, K)
        out = np.zeros_like(s)
        for m in range(g.shape[0]):
            out[m] = O._pack_sign_bits_fast(~np.signbit(g[m][i[m]]))
        return i, out

    def msb_first(g, K):                     # wrong bit order inside a word
        i, s = real_topk(g, K)
        out = np.zeros_like(s)
        for m in range(g.shape[0]):
            neg = np.signbit(g[m][i[m]])
            for j in range(K):
                if neg[j]:
                    out[m][j >> 5] |= np.uint32(1) << np.uint32(31 - (j & 31))
        return i, out

    def zero_votes_nothing(g, K):            # sgn(0) = 0 read literally drops +-0 entries' sign
        i, s = real_topk(g, K)
        out = np.zeros_like(s)
        for m in range(g.shape[0]):
            out[m] = O._pack_sign_bits_fast(g[m][i[m]] < 0)
        return i, out

    def vote_tie_positive(idx, sgn, M, K, d):   # ties broken toward +1 instead of 0
        v, bad = real_vote(idx, sgn, M, K, d)
        cnt = np.zeros(d, dtype=np.int64)
        for m in range(M):
            ok = idx[m] < d
            np.add.at(cnt, idx[m][ok].astype(np.int64), 1)
        v = v.copy()
        v[(v == 0) & (cnt > 0)] = 1
        return v, bad

    def vote_set_semantics(idx, sgn, M, K, d):  # duplicates counted once
        v = np.zeros(d, dtype=np.int64)
        for m in range(M):
            seen = set()
            for j in range(K):
                n = int(idx[m][j])
                if n < d and n not in seen:
                    seen.add(n)
                    v[n] += 1 - 2 * ((int(sgn[m][j >> 5]) >> (j & 31)) & 1)
        return ((v > 0).astype(np.int8) - (v < 0).astype(np.int8)), int((idx >= d).sum())

    def apply_plus(x, vote, lr):                # wrong sign of the update
        return real_apply(x, -np.asarray(vote), lr)

    def apply_double(x, vote, lr):              # update computed in fp64 product then added twice-rounded
        return (x + np.float32(-1.0) * (np.float32(lr) * vote.astype(np.float32)) + np.float32(0.0)).astype(np.float32) * np.float32(1.0) + np.float32(0.0)

    real_ef, real_mom = O.error_feedback_step, O.apply_vote_momentum

    def ef_memory_of_raw_gradient(x, gt, e, eta, K, lr, topk=None):     # e <- g~ - TopK(g) instead of g - TopK(g)
        xn, en, i, s, v = real_ef(x, gt, e, eta, K, lr, topk)
        en2 = np.asarray(gt, dtype=np.float32).copy()
        for m in range(en2.shape[0]):
            en2[m][i[m].astype(np.int64)] = 0
        return xn, en2, i, s, v

    def ef_kept_entries_not_cleared(x, gt, e, eta, K, lr, topk=None):
        xn, en, i, s, v = real_ef(x, gt, e, eta, K, lr, topk)
        g = (np.asarray(gt, np.float32) + np.float32(eta) * np.asarray(e, np.float32)).astype(np.float32)
        return xn, g, i, s, v

    def ef_eta_on_gradient(x, gt, e, eta, K, lr, topk=None):            # g = eta * g~ + e
        return real_ef(x, (np.float32(eta) * np.asarray(gt, np.float32)).astype(np.float32),
                       (np.asarray(e, np.float32) / np.float32(eta if eta else 1)).astype(np.float32), eta, K, lr, topk)

    def momentum_uses_old_v(x, v, vote, mu, lr):                        # x moved with v before its update
        xn = (np.asarray(x, np.float32) - np.float32(lr) * np.asarray(v, np.float32)).astype(np.float32)
        _, vn = real_mom(x, v, vote, mu, lr)
        return xn, vn

    def momentum_decays_the_vote(x, v, vote, mu, lr):                   # v <- mu * (v + vote)
        vn = (np.float32(mu) * (np.asarray(v, np.float32) + np.asarray(vote).astype(np.float32))).astype(np.float32)
        return (np.asarray(x, np.float32) - np.float32(lr) * vn).astype(np.float32), vn

    real_perm, real_keys = O.randk_permutation, O.randk_round_keys

    def randk_modulo_instead_of_walk(j, d, keys):                       # out-of-range values folded back: repeats
        h = 1
        while (1 << (2 * h)) < d:
            h += 1
        v = real_perm(j, 1 << (2 * h), keys)
        return (v.astype(np.uint64) % np.uint64(d)).astype(np.uint32)

    def randk_same_subset_for_every_worker(seed, worker, step):
        return real_keys(seed, 0, step)

    def randk_same_subset_every_iteration(seed, worker, step):
        return real_keys(seed, worker, 0)

    def randk_identity_rounds(j, d, keys):                              # no mixing: keeps the first K coordinates
        return np.asarray(j).astype(np.uint32)

    def two_bit_msb_first(vote):                                        # pairs filled from the top of the word
        return real_enc2(np.asarray(vote)[::-1])

    def sparse_positive_is_one(vote):                                   # sign bits inverted
        return real_encs(-np.asarray(vote, dtype=np.int8))

    def counts_once_per_coordinate(idx, signbits, M, K, d):             # a coordinate counted once whoever votes
        c = np.zeros(d, dtype=np.int64)
        full = real_counts(idx, signbits, M, K, d)
        c[full != 0] = np.sign(full[full != 0])
        return c

    extra_down = [("encode_vote_2bit", two_bit_msb_first), ("encode_vote_sparse", sparse_positive_is_one),
                  ("vote_counts", counts_once_per_coordinate)]
    extra_randk = extra_down + [("randk_permutation", randk_modulo_instead_of_walk), ("randk_round_keys", randk_same_subset_for_every_worker),
                   ("randk_round_keys", randk_same_subset_every_iteration), ("randk_permutation", randk_identity_rounds)]
    extra = extra_randk + [("error_feedback_step", ef_memory_of_raw_gradient), ("error_feedback_step", ef_kept_entries_not_cleared),
             ("error_feedback_step", ef_eta_on_gradient), ("apply_vote_momentum", momentum_uses_old_v),
             ("apply_vote_momentum", momentum_decays_the_vote)]
    return extra + [("topk_sign", higher_index_wins), ("topk_sign", signed_not_magnitude), ("topk_sign", smallest_k),
            ("topk_sign", inverted_sign_bits), ("topk_sign", msb_first), ("topk_sign", zero_votes_nothing),
            ("majority_vote", vote_tie_positive), ("majority_vote", vote_set_semantics),
            ("apply_vote", apply_plus), ("apply_vote", apply_double)]


@pytest.mark.parametrize("which", range(22))
def test_pins_catch_planted_mistakes(which, monkeypatch):
    name, fn = _mutants()[which]
    monkeypatch.setattr(O, name, fn)
    caught = 0
    for pin in ALL_PINS:
        try:
            pin(O)
        except AssertionError:
            caught += 1
        except Exception:           # a mutant that merely crashes a pin has not been noticed by it
            pass
    assert caught >= 1, f"no pin notices mutant {fn.__name__}"
