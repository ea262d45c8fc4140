"""Pins for the oracle's suffix-match search and draft gather (Sec. 3.1, 3.2; App. B.3
step 1).  None of these re-type the scan: they use exhaustive enumeration, closed
forms, the paper's hash-map method written separately, and planted ground truth."""
import itertools

import numpy as np
import pytest

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import inputs


def _definition(h, n, g):
    """The definition, spelled out with Python slices only."""
    if n < 2 * g:
        return []
    key = list(h[n - g:n])
    return [p for p in range(0, n - 2 * g + 1) if list(h[p:p + g]) == key]


@pytest.mark.parametrize("vocab,nmax", [(2, 11), (3, 8)])
def test_exhaustive_small_strings(vocab, nmax):
    for n in range(1, nmax + 1):
        for h in itertools.product(range(vocab), repeat=n):
            h = np.array(h, dtype=np.int32)
            for g in range(1, 6):
                want = _definition(h, n, g)
                assert O.all_matches_bruteforce(h, n, g) == want
                assert O.find_match(h, n, g, O.LATEST) == (want[-1] if want else -1)
                assert O.find_match(h, n, g, O.FIRST) == (want[0] if want else -1)


def test_random_small_alphabet_against_enumeration():
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.integers(1, 33))
        h = rng.integers(0, 4, size=n, dtype=np.int32)
        for g in range(1, 6):
            want = _definition(h, n, g)
            assert O.find_match(h, n, g, O.LATEST) == (want[-1] if want else -1)
            assert O.find_match(h, n, g, O.FIRST) == (want[0] if want else -1)


@pytest.mark.parametrize("n", [6, 7, 50, 1001])
@pytest.mark.parametrize("g", [1, 3, 5])
def test_closed_form_constant_history(n, g):
    h = np.full(n, 7, dtype=np.int32)
    if n < 2 * g:
        assert O.find_match(h, n, g, O.LATEST) == -1
        return
    assert O.find_match(h, n, g, O.LATEST) == n - 2 * g       # last non-overlapping start
    assert O.find_match(h, n, g, O.FIRST) == 0


def test_closed_form_increasing_history_has_no_match():
    h = np.arange(500, dtype=np.int32)
    for g in (1, 3, 5):
        assert O.find_match(h, 500, g, O.LATEST) == -1
        assert O.find_match(h, 500, g, O.FIRST) == -1


@pytest.mark.parametrize("P,n,g", [(7, 100, 3), (5, 23, 5), (11, 64, 3), (4, 9, 3), (9, 17, 3)])
def test_closed_form_periodic_history(P, n, g):
    h = (np.arange(n) % P).astype(np.int32)
    # with P >= g every window is determined by its first element's phase
    phase = (n - g) % P
    starts = [p for p in range(phase, n - 2 * g + 1, P)]
    assert O.find_match(h, n, g, O.LATEST) == (starts[-1] if starts else -1)
    assert O.find_match(h, n, g, O.FIRST) == (starts[0] if starts else -1)


def test_too_short_and_degenerate():
    h = np.array([1, 2, 3, 1, 2], dtype=np.int32)
    assert O.find_match(h, 5, 3, O.LATEST) == -1          # n < 2*gamma
    assert O.find_match(h, 0, 3, O.LATEST) == -1
    assert O.find_match(h, 5, 0, O.LATEST) == -1
    # overlap with the key itself is not a match (App. B.3 step 1(c))
    h = np.array([5, 5, 5, 5, 5], dtype=np.int32)
    assert O.find_match(h, 5, 3, O.LATEST) == -1
    h = np.array([5, 5, 5, 5, 5, 5], dtype=np.int32)
    assert O.find_match(h, 6, 3, O.LATEST) == 0


def test_dictionary_method_agrees():
    """Sec. 3.1: hash map of all gamma-grams, O(gamma) insert and lookup per token."""
    rng = np.random.default_rng(3)
    for g in (1, 2, 3, 5):
        for vocab in (3, 50):
            d = O.GammaGramDict(g)
            h = []
            for _ in range(200):
                t = int(rng.integers(0, vocab))
                d.append(t)
                h.append(t)
                arr = np.asarray(h, dtype=np.int32)
                for pol in (O.LATEST, O.FIRST):
                    assert d.lookup(pol) == O.find_match(arr, len(h), g, pol)


def test_planted_span_ground_truth():
    """Uniform ids over a large vocabulary: the planted copy is the only repeat, so
    the search must return the span's source and the draft must be its continuation."""
    rng = np.random.default_rng(5)
    n, vocab = 4000, 1 << 30
    for _ in range(20):
        h = rng.integers(0, vocab, size=n).astype(np.int64)
        spans = inputs.plant_repeats(rng, h, 4, 40, 40, limit=n - 64)
        src, dst, ln = spans[int(rng.integers(0, 4))]
        t = int(rng.integers(3, 30))
        cut = dst + t                      # history ends t tokens into the replayed span
        for g in (3,):
            p0 = O.find_match(h, cut, g, O.LATEST)
            assert p0 == src + t - g
            assert O.find_match(h, cut, g, O.FIRST) == p0
            draft = O.gather_draft(h, cut, p0, g, 10)
            assert draft == [int(x) for x in h[src + t:src + t + 10]]


def test_gather_clips_at_history_end():
    h = np.array([9, 1, 2, 3, 4, 8, 1, 2, 3], dtype=np.int32)
    p0 = O.find_match(h, 9, 3, O.LATEST)
    assert p0 == 1
    assert O.gather_draft(h, 9, p0, 3, 10) == [4, 8, 1, 2, 3]   # only 5 tokens follow
    assert O.gather_draft(h, 9, p0, 3, 2) == [4, 8]
    assert O.gather_draft(h, 9, -1, 3, 10) == []
    # the draft length is at least gamma whenever a match exists (non-overlap)
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(6, 40))
        hh = rng.integers(0, 3, size=n, dtype=np.int32)
        p = O.find_match(hh, n, 3, O.LATEST)
        if p >= 0:
            assert len(O.gather_draft(hh, n, p, 3, 10)) >= 3


def test_search_workload_shapes():
    hist, kinds, spans = inputs.match_search_histories(batch=8, n=4096, n_spans=4,
                                                       span_lo=64, span_hi=256)
    assert hist.shape == (8, 4096) and hist.dtype == np.int32
    for b in range(8):
        for g in (3, 5):
            p = O.find_match(hist[b], 4096, g, O.LATEST)
            if kinds[b] in (0, 1):
                assert p >= 0          # the tail replays a planted span
            if kinds[b] == 3:
                assert p == -1         # reserved id never occurs earlier
