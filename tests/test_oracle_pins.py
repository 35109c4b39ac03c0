"""Pins for the CPU oracle: it is checked against things other than itself --
an exhaustive shortest-path search over single-symbol edits, closed forms,
metric invariants, the extreme values the paper states for d_K, exact rational
arithmetic, closed-form z-scores and an independent library routine."""
import itertools
import math
import os
from collections import deque
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- edit distance
def _neighbours(s, alphabet, max_len):
    for i in range(len(s)):
        yield s[:i] + s[i + 1:]                       # delete
        for c in alphabet:
            if c != s[i]:
                yield s[:i] + (c,) + s[i + 1:]        # substitute
    if len(s) < max_len:
        for i in range(len(s) + 1):
            for c in alphabet:
                yield s[:i] + (c,) + s[i:]            # insert


def _edit_graph_distances(src, alphabet, max_len):
    """Fewest single-symbol insertions/deletions/substitutions from ``src`` to every
    string of length <= max_len: breadth-first search over the edit graph, i.e.
    the definition of Levenshtein distance, with no dynamic programme."""
    dist = {src: 0}
    q = deque([src])
    while q:
        s = q.popleft()
        for t in _neighbours(s, alphabet, max_len):
            if t not in dist:
                dist[t] = dist[s] + 1
                q.append(t)
    return dist


@pytest.mark.parametrize("alphabet,max_len", [((0, 1), 5), ((0, 1, 2), 4)])
def test_levenshtein_matches_edit_graph_search(alphabet, max_len):
    strings = [t for L in range(max_len + 1) for t in itertools.product(alphabet, repeat=L)]
    for src in strings:
        # intermediate strings of an optimal script never need to exceed the longer
        # endpoint, so a search bounded by max_len is exact for targets <= max_len
        ref = _edit_graph_distances(src, alphabet, max_len)
        for dst in strings:
            assert oracle.levenshtein(src, dst) == ref[dst], (src, dst)


def _rec(a, b):
    if not a:
        return len(b)
    if not b:
        return len(a)
    return min(_rec(a[1:], b) + 1, _rec(a, b[1:]) + 1, _rec(a[1:], b[1:]) + (a[0] != b[0]))


def test_levenshtein_matches_exponential_recursion():
    rng = np.random.default_rng(11)
    for _ in range(300):
        m, n = rng.integers(0, 7, size=2)
        a = tuple(int(x) for x in rng.integers(0, 3, size=m))
        b = tuple(int(x) for x in rng.integers(0, 3, size=n))
        assert oracle.levenshtein(a, b) == _rec(a, b)


def test_levenshtein_textbook_fixture():
    with open(os.path.join(GOLDEN, "levenshtein_textbook.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 8
    for ln in rows:
        a, b, d = [x.strip() for x in ln.split(";")]
        assert oracle.levenshtein([ord(c) for c in a], [ord(c) for c in b]) == int(d), ln


def test_levenshtein_closed_forms():
    rng = np.random.default_rng(5)
    for _ in range(50):
        m = int(rng.integers(1, 60))
        a = rng.integers(-2 ** 31, 2 ** 31 - 1, size=m)
        assert oracle.levenshtein(a, a) == 0
        assert oracle.levenshtein(a, []) == m
        assert oracle.levenshtein([], a) == m
        n = int(rng.integers(1, 60))
        b = rng.integers(0, 1000, size=n) + 10 ** 6          # disjoint alphabet
        a2 = rng.integers(0, 1000, size=m)
        assert oracle.levenshtein(a2, b) == max(m, n)
        k = int(rng.integers(0, m))
        sub = a.copy()
        sub[k] = sub[k] ^ 1
        assert oracle.levenshtein(a, sub) == 1
        assert oracle.levenshtein(a, np.delete(a, k)) == 1
        assert oracle.levenshtein(a, np.insert(a, k, a[k] ^ 1)) == 1
    # a transposition costs two unit edits (no transposition operation)
    assert oracle.levenshtein([1, 2], [2, 1]) == 2
    # shifting by one position costs 2 (delete front, insert back), not the Hamming distance
    assert oracle.levenshtein([1, 2, 3, 4, 5, 6], [2, 3, 4, 5, 6, 7]) == 2


def test_levenshtein_invariants():
    rng = np.random.default_rng(7)
    for _ in range(200):
        la, lb, lc = rng.integers(0, 40, size=3)
        v = int(rng.integers(2, 6))
        a, b, c = (rng.integers(0, v, size=L) for L in (la, lb, lc))
        dab, dba = oracle.levenshtein(a, b), oracle.levenshtein(b, a)
        assert dab == dba
        assert abs(int(la) - int(lb)) <= dab <= max(la, lb)
        assert oracle.levenshtein(a, c) <= dab + oracle.levenshtein(b, c)
        if la == lb:
            assert dab <= int((a != b).sum())
        # asymmetric operands: a transposed DP would still be symmetric, so also pin
        # the prefix property d(a, a + tail) == len(tail)
        tail = rng.integers(10, 20, size=int(rng.integers(0, 9)))
        assert oracle.levenshtein(a, np.concatenate([a, tail])) == tail.size


# ------------------------------------------------------------------------- d_K
def _parse_group(text):
    rows = [[int(x) for x in r.split(",")] for r in text.split("|")]
    return np.array(rows, dtype=np.int32)


def test_dk_extremes_from_paper():
    with open(os.path.join(GOLDEN, "dk_extremes.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for ln in rows:
        name, G, K, body, want = [x.strip() for x in ln.split(";")]
        grp = _parse_group(body)
        assert grp.shape == (int(G), int(K))
        seqs = np.zeros((1, int(G), 8), dtype=np.int32)
        seqs[0, :, :int(K)] = grp
        _, _, mean, _ = oracle.gate(seqs, None, int(K), 0.12)
        assert mean[0] == float(want), name


def test_dk_range_normalisation_and_order():
    rng = np.random.default_rng(3)
    G, N, S = 40, 5, 16
    seqs = rng.integers(0, 4, size=(G, N, S)).astype(np.int32)
    lens = rng.integers(0, S + 1, size=(G, N)).astype(np.int32)
    K = 12
    pd, ps, mean, stop = oracle.gate(seqs, lens, K, 0.5)
    assert ((mean >= 0) & (mean <= 1)).all()
    m = np.minimum(lens, K)
    for g in range(G):
        p = 0
        terms = []
        for i in range(N):
            for j in range(i + 1, N):
                # the pair order and the operands of every entry, from single calls
                d = oracle.levenshtein(seqs[g, i, :m[g, i]], seqs[g, j, :m[g, j]])
                assert pd[g, p] == d
                longer = max(m[g, i], m[g, j])
                terms.append(Fraction(d, int(longer)) if longer else Fraction(0))
                p += 1
        assert ps[g] == pd[g].sum()
        exact = sum(terms) / len(terms)
        assert abs(mean[g] - float(exact)) <= 4e-16 * len(terms)
        assert stop[g] == (mean[g] < 0.5)


def test_dk_normalises_by_longer_prefix_and_empty_pairs():
    seqs = np.zeros((1, 3, 8), dtype=np.int32)
    seqs[0, 0, :4] = [1, 2, 3, 4]
    seqs[0, 1, :2] = [1, 2]
    lens = np.array([[4, 2, 0]], dtype=np.int32)
    pd, ps, mean, _ = oracle.gate(seqs, lens, 8, 0.1)
    assert pd.tolist() == [[2, 4, 2]]
    # (2/4 + 4/4 + 2/2) / 3
    assert mean[0] == pytest.approx((0.5 + 1.0 + 1.0) / 3, abs=1e-15)
    lens0 = np.zeros((1, 3), dtype=np.int32)
    _, _, mean0, stop0 = oracle.gate(seqs, lens0, 8, 0.1)
    assert mean0[0] == 0.0 and stop0[0] == 1
    # prefix truncation at K: only the first K actions count
    lensK = np.array([[4, 4, 4]], dtype=np.int32)
    seqs[0, 1, :4] = [1, 2, 9, 9]
    seqs[0, 2, :4] = [1, 2, 8, 8]
    _, _, meanK, _ = oracle.gate(seqs, lensK, 2, 0.1)
    assert meanK[0] == 0.0
    # raw mode reports the un-normalised mean distance
    pd4, ps4, mean4, _ = oracle.gate(seqs, lensK, 4, 0.1, oracle.NORM_NONE)
    assert mean4[0] == pytest.approx(ps4[0] / 3.0, abs=1e-15)


def test_gate_is_strict_and_monotone_in_threshold():
    seqs = np.zeros((1, 2, 4), dtype=np.int32)
    seqs[0, 0] = [1, 2, 3, 4]
    seqs[0, 1] = [1, 2, 3, 5]                       # d = 1, longer = 4 -> d_K = 0.25 exactly
    _, _, mean, stop = oracle.gate(seqs, None, 4, 0.25)
    assert mean[0] == 0.25 and stop[0] == 0          # Eq. 2 is a strict inequality
    _, _, _, stop = oracle.gate(seqs, None, 4, math.nextafter(0.25, 1.0))
    assert stop[0] == 1
    rng = np.random.default_rng(9)
    seqs = rng.integers(0, 3, size=(200, 4, 12)).astype(np.int32)
    prev = np.zeros(200, dtype=np.uint8)
    # cut sets are nested as the threshold grows (Table 1 sweeps d_L upward)
    for thr in [0.0, 0.05, 0.08, 0.10, 0.12, 0.14, 0.18, 0.5, 1.0, 1.5]:
        _, _, mean, stop = oracle.gate(seqs, None, 12, thr)
        assert (stop >= prev).all()
        prev = stop
        if thr == 0.0:
            assert stop.sum() == 0
        if thr > 1.0:
            assert stop.sum() == 200


def test_exact_rational_mask_agrees_away_from_the_edge():
    rng = np.random.default_rng(21)
    seqs = rng.integers(0, 3, size=(300, 4, 10)).astype(np.int32)
    lens = rng.integers(1, 11, size=(300, 4)).astype(np.int32)
    pd, _, mean, stop = oracle.gate(seqs, lens, 10, 0.4)
    exact = oracle.exact_mask(pd, lens, 10, 0.4)
    far = np.abs(mean - 0.4) > 1e-12
    assert (stop[far] == exact[far]).all()


def test_threads_do_not_change_results():
    rng = np.random.default_rng(2)
    seqs = rng.integers(0, 5, size=(37, 6, 20)).astype(np.int32)
    lens = rng.integers(0, 21, size=(37, 6)).astype(np.int32)
    one = oracle.gate(seqs, lens, 17, 0.3, threads=1)
    many = oracle.gate(seqs, lens, 17, 0.3, threads=4)
    for x, y in zip(one, many):
        assert np.array_equal(x, y)


def test_stream_replay_recomputes_from_scratch():
    A = oracle.NO_ACTION
    actions = np.array([[[1, 1]], [[2, 3]], [[A, 4]]], dtype=np.int32)   # steps x 1 group x 2
    out = list(oracle.gate_stream(actions, 0.3))
    assert [int(o[1][0, 0]) for o in out] == [0, 1, 2]
    # after step 3 the prefixes are [1,2] and [1,3,4]: d = 2, longer = 3
    assert out[2][3][0] == pytest.approx(2 / 3, abs=1e-15)
    assert [int(o[4][0]) for o in out] == [1, 0, 0]


# ------------------------------------------------------------------ advantages
def test_advantage_binary_closed_form():
    eps = 1e-6
    for N in (2, 5, 8, 16):
        for s in range(1, N):
            r = np.zeros((1, N), dtype=np.float32)
            r[0, :s] = 1.0
            adv, zv = oracle.advantage(r, None, eps)
            p = s / N
            sigma = math.sqrt(p * (1 - p))
            e = float(np.float32(eps))
            assert zv[0] == 0
            assert adv[0, 0] == pytest.approx((1 - p) / (sigma + e), rel=1e-6)
            assert adv[0, -1] == pytest.approx(-p / (sigma + e), rel=1e-6)
            assert adv[0, 0] > 0 > adv[0, -1]


def test_advantage_identities_and_population_std():
    import torch
    rng = np.random.default_rng(4)
    r = rng.random((64, 8)).astype(np.float32)
    eps = 1e-6
    adv, zv = oracle.advantage(r, None, eps)
    assert not zv.any()
    r64 = torch.from_numpy(r).double()
    sigma = torch.std(r64, dim=1, unbiased=False).numpy()      # 1/G, not 1/(G-1)
    mean = r64.mean(dim=1).numpy()
    want = (r.astype(np.float64) - mean[:, None]) / (sigma[:, None] + float(np.float32(eps)))
    assert np.allclose(adv, want, rtol=1e-6, atol=0)
    assert np.abs(adv.astype(np.float64).sum(axis=1)).max() < 1e-5
    ssq = (adv.astype(np.float64) ** 2).sum(axis=1)
    assert np.allclose(ssq, 8 * sigma ** 2 / (sigma + 1e-6) ** 2, rtol=1e-5)
    # with the sample (1/(G-1)) normaliser the values would differ by sqrt(8/7)
    wrong = torch.std(r64, dim=1, unbiased=True).numpy()
    assert not np.allclose(sigma, wrong, rtol=1e-3)


def test_zero_variance_and_dropped_groups_are_exact_zeros():
    r = np.array([[0.3] * 8, [1.0] * 8, [0.0] * 8, [0.0, -0.0] * 4,
                  [0.1, 0.2, 0.3, 0.4, 0.5, 0.6, 0.7, 0.8]], dtype=np.float32)
    adv, zv = oracle.advantage(r, None, 1e-6)
    assert zv.tolist() == [1, 1, 1, 1, 0]
    assert (adv[:4] == 0).all() and not np.signbit(adv[:4]).any()
    drop = np.array([0, 0, 0, 0, 1], dtype=np.uint8)
    adv2, zv2 = oracle.advantage(r, drop, 1e-6)
    assert (adv2 == 0).all() and not np.signbit(adv2).any()
    assert zv2.tolist() == [1, 1, 1, 1, 0]           # the flag still reflects the rewards
    # 0.3f repeated: the fp64 mean of equal values need not round-trip, the flag must not care
    r3 = np.full((1, 7), np.float32(0.3), dtype=np.float32)
    adv3, zv3 = oracle.advantage(r3, None, 0.0)
    assert zv3[0] == 1 and (adv3 == 0).all()
    # NaN equals nothing: not zero-variance, NaN propagates
    rn = np.array([[np.nan, 1, 1, 1]], dtype=np.float32)
    advn, zvn = oracle.advantage(rn, None, 1e-6)
    assert zvn[0] == 0 and np.isnan(advn).all()


def test_advantage_eps_zero_gives_unit_variance():
    rng = np.random.default_rng(8)
    r = rng.random((32, 16)).astype(np.float32)
    adv, _ = oracle.advantage(r, None, 0.0)
    a = adv.astype(np.float64)
    assert np.allclose((a ** 2).mean(axis=1), 1.0, rtol=1e-5)
