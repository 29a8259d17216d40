"""Pins for the oracle's SCORE (Eq. 1, bitcount-xor identity) and TOPK (standard top-k, ties to
the lowest index): hand-derived fixtures, bit-level brute force, the O(n^2) rank definition and
invariants.  CPU only."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def test_golden_hamming_cases():
    for ln in _lines("hamming_cases.txt"):
        qc, kc, ham, sc = ln.split()
        s = oracle.score([int(qc, 16)], [int(kc, 16)])
        assert int(s[0]) == int(sc) == 32 - int(ham), ln


def test_score_equals_32_minus_bitwise_hamming_brute_force():
    rng = np.random.default_rng(10)
    q = rng.integers(0, 2**32, size=1, dtype=np.uint64).astype(np.uint32)
    k = rng.integers(0, 2**32, size=5000, dtype=np.uint64).astype(np.uint32)
    s = oracle.score(q, k)
    qb = np.unpackbits(q.view(np.uint8)).reshape(1, 32)
    kb = np.unpackbits(k.view(np.uint8)).reshape(-1, 32)
    ham = (qb != kb).sum(axis=1)
    assert np.array_equal(s, 32 - ham)
    assert s.min() >= 0 and s.max() <= 32
    # library popcount of the xor
    assert np.array_equal(s, 32 - np.array([bin(int(a) ^ int(q[0])).count("1") for a in k]))


def test_score_special_values_and_invariances():
    rng = np.random.default_rng(11)
    k = rng.integers(0, 2**32, size=1000, dtype=np.uint64).astype(np.uint32)
    q = np.uint32(0x9E3779B9)
    assert np.all(oracle.score([q], [q]) == 32)
    assert np.all(oracle.score([q], [~q]) == 0)
    base = oracle.score([q], k)
    mask = np.uint32(0xC0FFEE11)
    assert np.array_equal(oracle.score([q ^ mask], k ^ mask), base)       # common flip mask
    rot = lambda v: ((v << np.uint32(7)) | (v >> np.uint32(25))).astype(np.uint32)
    assert np.array_equal(oracle.score([rot(np.array([q]))[0]], rot(k)), base)   # common bit permutation
    # Hamming distance is symmetric in its two arguments
    assert all(int(oracle.score([kk], [q])[0]) == int(b) for kk, b in zip(k[:50], base[:50]))


def test_group_score_is_max_over_group_and_reduces_to_eq1_for_one_head():
    rng = np.random.default_rng(12)
    k = rng.integers(0, 2**32, size=3000, dtype=np.uint64).astype(np.uint32)
    qs = rng.integers(0, 2**32, size=4, dtype=np.uint64).astype(np.uint32)
    per_head = np.stack([oracle.score([qq], k) for qq in qs])
    assert np.array_equal(oracle.score(qs, k), per_head.max(axis=0))
    assert np.array_equal(oracle.score(qs[:1], k), per_head[0])
    assert np.array_equal(oracle.score(qs[[2, 0, 3, 1]], k), oracle.score(qs, k))


def test_golden_topk_cases():
    for ln in _lines("topk_cases.txt"):
        k, scores, sel = [p.strip() for p in ln.split("|")]
        got = oracle.topk([int(v) for v in scores.split()], int(k))
        assert got.tolist() == [int(v) for v in sel.split()], ln


def test_golden_topk_window_cases():
    for ln in _lines("topk_window_cases.txt"):
        k, n_sink, n_local, scores, sel = [p.strip() for p in ln.split("|")]
        got = oracle.topk_windows([int(v) for v in scores.split()], int(k), int(n_sink), int(n_local))
        assert got.tolist() == [int(v) for v in sel.split()], ln


def _window_definition(scores, k, n_sink, n_local):
    """Written from the sentence, not from the code: always-kept tokens, then rank among the others."""
    n = len(scores)
    forced = [i for i in range(n) if i < n_sink or i >= n - n_local]
    others = [i for i in range(n) if i not in forced]
    heavy = []
    for i in others:
        better = sum(1 for j in others if scores[j] > scores[i] or (scores[j] == scores[i] and j < i))
        if better < k:
            heavy.append(i)
    return sorted(forced + heavy)


@pytest.mark.parametrize("seed", range(6))
def test_topk_windows_matches_its_definition_and_reduces_to_plain_topk(seed):
    rng = np.random.default_rng(300 + seed)
    for n in (1, 2, 7, 33, 64):
        scores = rng.integers(12, 22, size=n)           # narrow range -> heavy ties
        for k in (0, 1, n // 2, n):
            assert oracle.topk_windows(scores, k, 0, 0).tolist() == oracle.topk(scores, k).tolist()
            for n_sink, n_local in ((1, 0), (0, 1), (2, 3), (n // 2, n // 2), (n, 0), (n + 2, n + 2), (5, 40)):
                got = oracle.topk_windows(scores, k, n_sink, n_local).tolist()
                assert got == _window_definition(scores.tolist(), k, n_sink, n_local), (n, k, n_sink, n_local)


def test_topk_windows_properties_on_large_input():
    rng = np.random.default_rng(9)
    n, k, n_sink, n_local = 50000, 1500, 128, 128
    scores = rng.integers(14, 24, size=n)
    sel = oracle.topk_windows(scores, k, n_sink, n_local)
    assert len(sel) == n_sink + n_local + k and np.all(np.diff(sel) > 0)
    assert set(range(n_sink)) <= set(sel.tolist()) and set(range(n - n_local, n)) <= set(sel.tolist())
    heavy = np.array(sorted(set(sel.tolist()) - set(range(n_sink)) - set(range(n - n_local, n))))
    middle = scores[n_sink:n - n_local]
    assert np.array_equal(heavy - n_sink, oracle.topk(middle, k))   # plain top-k of the tokens in between


def _rank_definition(scores, k):
    n = len(scores)
    sel = []
    for i in range(n):
        better = sum(1 for j in range(n) if scores[j] > scores[i] or (scores[j] == scores[i] and j < i))
        if better < k:
            sel.append(i)
    return sel


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_rank_definition_on_small_inputs(seed):
    rng = np.random.default_rng(100 + seed)
    for n in (1, 2, 7, 33, 64):
        scores = rng.integers(12, 22, size=n)           # narrow range -> heavy ties
        for k in (0, 1, n // 2, n - 1, n, n + 3):
            assert oracle.topk(scores, k).tolist() == _rank_definition(scores.tolist(), k)


def test_topk_properties_on_large_tied_input():
    rng = np.random.default_rng(13)
    n = 20000
    scores = np.clip(np.rint(rng.normal(18, 1.8, size=n)), 0, 32).astype(np.int32)
    prev = set()
    for k in (1, 50, 625, 626, 5000, n):
        idx = oracle.topk(scores, k)
        assert len(idx) == min(k, n) and np.all(np.diff(idx) > 0)
        sel = np.zeros(n, bool)
        sel[idx] = True
        if k < n:
            t = scores[sel].min()
            assert t >= scores[~sel].max()
            tied_sel = np.nonzero(sel & (scores == t))[0]
            tied_not = np.nonzero(~sel & (scores == t))[0]
            if len(tied_sel) and len(tied_not):
                assert tied_sel.max() < tied_not.min()
        assert prev <= set(idx.tolist())                 # nesting I_k subset I_k'
        prev = set(idx.tolist())
    # library sort: lexsort by (index asc) within (score desc)
    order = np.lexsort((np.arange(n), -scores))
    assert sorted(order[:625].tolist()) == oracle.topk(scores, 625).tolist()
    assert np.bincount(scores, minlength=33).sum() == n


def test_topk_all_equal_scores_takes_lowest_indices():
    assert oracle.topk(np.full(100, 17), 10).tolist() == list(range(10))
    assert oracle.topk(np.full(5, 0), 10).tolist() == list(range(5))
    assert oracle.topk(np.array([], dtype=np.int32), 4).tolist() == []


def test_unpaging_signatures_is_storage_only():
    """A paged signature cache read back through its block table gives the signatures that were put in, whatever the
    page order and page size, so scores and selections over it are those over the contiguous cache."""
    rng = np.random.default_rng(15)
    n, Hkv = 75, 3
    codes = rng.integers(0, 2**32, size=(Hkv, n), dtype=np.uint64).astype(np.uint32)
    q = rng.integers(0, 2**32, size=2, dtype=np.uint64).astype(np.uint32)
    for ps in (1, 4, 16, 64):
        n_pages = (n + ps - 1) // ps
        perm = rng.permutation(n_pages + 4)[:n_pages]                 # pages scattered over a larger pool
        pool = np.full((n_pages + 4, Hkv, ps), 0xDEADBEEF, np.uint32)
        for t in range(n):
            pool[perm[t // ps], :, t % ps] = codes[:, t]
        for h in range(Hkv):
            back = oracle.unpage_codes(pool, perm, ps, h, n)
            assert np.array_equal(back, codes[h])
            assert np.array_equal(oracle.topk(oracle.score(q, back), 9), oracle.topk(oracle.score(q, codes[h]), 9))
        assert np.array_equal(oracle.unpage_codes(pool, perm, ps, 1, 10), codes[1, :10])   # a prefix of the sequence
