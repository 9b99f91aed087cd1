"""Pins of the oracle's proposal decoder (which move a Philox block names).

The move set is this build's reading of Section III-B for a schedule-valued state; what pins it is what its
definition and the mathematics fix: proposals decoded by hand from the published Philox known-answer blocks,
and the distribution of every field over many draws (shares, uniformity, independence), each with a chi-square
bound. A swapped pair of Philox words, an off-by-one in s0, a missing run-length class or a wrong swap share
turns at least one of these red; the planted-mistake cases at the end show that the statistics have that power.
"""
import os

import numpy as np
import pytest

GB = 10 ** 9
N = 200_000
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "proposal_worked.txt")


def _problem(oracle, U, S):
    A = np.zeros((S, (U + 31) // 32), np.uint32)
    return oracle.Problem(U, 8192, S, A, min(U, 3), 8 * GB, 1 * GB, 1 * GB)


def _draw(oracle, U, S, n=N, chain=7, seed=12345, tag=1, m_begin=0, **kw):
    prob = _problem(oracle, U, S)
    ap = prob.make_params(chains=chain + 1, moves=max(n, 1), seed=seed, **kw)
    return prob.decode_moves(ap, chain, m_begin, n, tag=tag).astype(np.int64)


def _chi2(counts, expected):
    counts = np.asarray(counts, np.float64)
    expected = np.asarray(expected, np.float64)
    return float(((counts - expected) ** 2 / expected).sum())


def _chi2_limit(dof):
    """Mean + 6 standard deviations of a chi-square variable with `dof` degrees of freedom: a correct decoder
    exceeds it with probability below 1e-6 for the dof used here, a biased one overshoots it by orders of magnitude."""
    return dof + 6.0 * (2.0 * dof) ** 0.5


def test_hand_decoded_proposals(oracle):
    rows = [l for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for line in rows:
        blk, shape, want = [part.split() for part in line.split("|")]
        ctr = [int(x, 16) for x in blk[:4]]
        key = [int(x, 16) for x in blk[4:]]
        S, U, p_swap, max_len = (int(x) for x in shape)
        prob = _problem(oracle, U, S)
        m = ctr[0] | (ctr[1] << 32)
        ap = prob.make_params(chains=1, moves=1, seed=key[0] | (key[1] << 32), p_swap_256=p_swap, max_len_log2=max_len)
        got = prob.decode_moves(ap, ctr[2], m, 1, tag=ctr[3])[0]
        assert [int(x) for x in got] == [int(x) for x in want], line


def test_swap_share(oracle):
    for p_swap in (0, 1, 77, 128, 255, 256):
        mv = _draw(oracle, 45, 37, p_swap_256=p_swap)
        k = int(mv[:, 0].sum())
        p = p_swap / 256.0
        if p in (0.0, 1.0):
            assert k == int(p * N)
        else:
            assert abs(k - N * p) < 6.0 * (N * p * (1 - p)) ** 0.5, p_swap


@pytest.mark.parametrize("max_len_log2,want", [(0, [1]), (1, [1, 2]), (3, [1, 2, 4, 8]), (5, [1, 2, 4, 8, 16, 30])])
def test_run_length_classes(oracle, max_len_log2, want):
    mv = _draw(oracle, 45, 37, max_len_log2=max_len_log2)
    vals, counts = np.unique(mv[:, 2], return_counts=True)
    assert list(vals) == want                                     # every class is drawn, no other length exists
    # the class is floor(byte * classes / 256): its share is the exact count of bytes that map to it
    share = np.bincount((np.arange(256) * len(want)) >> 8, minlength=len(want)) / 256.0
    if len(want) > 1:
        assert _chi2(counts, N * share) < _chi2_limit(len(want) - 1)


@pytest.mark.parametrize("S", [1, 2, 37, 100, 512, 1000, 32768])
def test_start_step_uniform_and_reaches_the_last_step(oracle, S):
    mv = _draw(oracle, 45, S)
    s0 = mv[:, 1]
    assert s0.min() == 0 and s0.max() <= S - 1
    if S <= 1000:
        assert s0.max() == S - 1                                  # the last step is proposed
        # s0 = floor(h * S / 65536) for a uniform 16-bit h: the exact share of every value
        share = np.bincount((np.arange(65536) * S) >> 16, minlength=S) / 65536.0
        if S > 1:
            assert _chi2(np.bincount(s0, minlength=S), N * share) < _chi2_limit(S - 1)
    else:
        # more steps than draws per bin allow: coarse bins, and both ends of the horizon are reached
        bins = np.bincount(s0 * 64 // S, minlength=64)
        assert _chi2(bins, np.full(64, N / 64.0)) < _chi2_limit(63)
        assert s0.max() > S - 1 - S // 1000


@pytest.mark.parametrize("U", [1, 2, 45, 256, 1000])
def test_units_uniform(oracle, U):
    mv = _draw(oracle, U, 37)
    for col in (3, 4):
        x = mv[:, col]
        assert x.min() == 0 and x.max() == U - 1
        if U > 1:
            assert _chi2(np.bincount(x, minlength=U), np.full(U, N / float(U))) < _chi2_limit(U - 1)


def test_large_unit_counts_are_covered(oracle):
    U = 2_621_440                                                 # more units than draws: coarse bins, both ends
    mv = _draw(oracle, U, 64)
    for col in (3, 4):
        x = mv[:, col]
        assert 0 <= x.min() < U // 1000 and U - U // 1000 < x.max() <= U - 1
        assert _chi2(np.bincount(x * 128 // U, minlength=128), np.full(128, N / 128.0)) < _chi2_limit(127)


def test_u_and_v_are_independent(oracle):
    U = 16
    mv = _draw(oracle, U, 37)
    u, v = mv[:, 3], mv[:, 4]
    same = int((u == v).sum())
    assert abs(same - N / U) < 6.0 * (N / U * (1 - 1 / U)) ** 0.5  # u == v at the rate 1/U, not 1 and not 0
    joint = np.bincount(u * U + v, minlength=U * U)
    assert _chi2(joint, np.full(U * U, N / float(U * U))) < _chi2_limit(U * U - 1)


def test_metropolis_uniform(oracle):
    mv = _draw(oracle, 45, 37)
    w = mv[:, 5]
    assert w.min() >= 0 and w.max() < 2 ** 32
    assert _chi2(np.bincount(w >> 24, minlength=256), np.full(256, N / 256.0)) < _chi2_limit(255)
    low = np.bincount(w & 255, minlength=256)                     # the low bits are random too
    assert _chi2(low, np.full(256, N / 256.0)) < _chi2_limit(255)
    assert abs(float(w.mean()) / 2 ** 32 - 0.5) < 6.0 / (12 * N) ** 0.5


def test_fields_are_pairwise_independent(oracle):
    """Every field against every other on coarse bins: swap, length class, s0 (three bit ranges of one Philox word),
    u, v and w (one word each)."""
    U, S = 64, 64
    mv = _draw(oracle, U, S)
    cls = {1: 0, 2: 1, 4: 2, 8: 3, 16: 4, 30: 5}
    f = {"swap": (mv[:, 0], 2), "len": (np.vectorize(cls.get)(mv[:, 2]), 6), "s0": (mv[:, 1] // 8, 8),
         "u": (mv[:, 3] // 8, 8), "v": (mv[:, 4] // 8, 8), "w": (mv[:, 5] >> 29, 8)}
    names = list(f)
    for i, a in enumerate(names):
        for b in names[i + 1:]:
            (xa, na), (xb, nb) = f[a], f[b]
            joint = np.bincount(xa * nb + xb, minlength=na * nb).reshape(na, nb).astype(np.float64)
            exp = joint.sum(1, keepdims=True) * joint.sum(0, keepdims=True) / joint.sum()
            assert _chi2(joint, exp) < _chi2_limit((na - 1) * (nb - 1)), (a, b)


def test_proposals_differ_between_chains_moves_seeds_and_tags(oracle):
    base = _draw(oracle, 1000, 100, n=2000)
    for other in (_draw(oracle, 1000, 100, n=2000, chain=8), _draw(oracle, 1000, 100, n=2000, seed=12346),
                  _draw(oracle, 1000, 100, n=2000, tag=2), _draw(oracle, 1000, 100, n=2000, m_begin=1 << 32)):
        assert (base[:, 5] == other[:, 5]).mean() < 0.01
    # move m of a long draw is the same proposal wherever the draw starts (pure function of the move index)
    shifted = _draw(oracle, 1000, 100, n=1000, m_begin=1000)
    assert np.array_equal(shifted, base[1000:])


def test_the_statistics_catch_planted_mistakes(oracle):
    """The same checks applied to deliberately wrong decodings of the oracle's own draws (the mistakes are planted
    here, on the CPU, in copies of the oracle's output)."""
    U, S = 16, 37
    mv = _draw(oracle, U, S)
    # v taken from the word u comes from: u == v always
    wrong_v = mv[:, 3]
    assert int((mv[:, 3] == wrong_v).sum()) - N / U > 6.0 * (N / U) ** 0.5
    # '<=' in place of '<' in the swap test: at p_swap_256 = 1 the share doubles, outside the bound of test_swap_share
    p = 1 / 256.0
    assert 2 * N * p - N * p > 6.0 * (N * p * (1 - p)) ** 0.5
    # s0 that never reaches the last step (S - 1 used in place of S)
    share = np.bincount((np.arange(65536) * S) >> 16, minlength=S) / 65536.0
    wrong = mv[:, 1] * (S - 1) // S
    assert _chi2(np.bincount(wrong, minlength=S), N * share) > 10 * _chi2_limit(S - 1)
    # a run-length class that is never drawn (class 5 folded into class 4)
    folded = np.where(mv[:, 2] == 30, 16, mv[:, 2])
    assert sorted(set(folded.tolist())) != [1, 2, 4, 8, 16, 30]
