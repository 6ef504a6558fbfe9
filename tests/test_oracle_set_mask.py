"""Pins for the oracle's table build, valid-set masks and member ranges.

The oracle builds a prefix tree by insertion; these tests compare it with what
the definitions fix, computed a different way: Python's built-in sort of tuples
(lexicographic, shorter-first), a scan over every member for the valid set
(Section 2.1), and the lower-bound characterisation of Section 3.2
("t_m is valid iff V_m is a prefix of the row the binary search lands on").
"""
import bisect
import itertools
import os

import numpy as np
import pytest

import oracle
from workloads import CONFIGS, make_set, scaled


def _csr(rows):
    tok = np.array([t for r in rows for t in r], dtype=np.int32)
    off = np.zeros(len(rows) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(r) for r in rows])
    return tok, off


def _rows_of(tok, off):
    return [tuple(int(x) for x in tok[off[i]:off[i + 1]]) for i in range(len(off) - 1)]


def _is_prefix(a, s):
    return len(a) <= len(s) and tuple(s[:len(a)]) == tuple(a)


def _brute_mask(members, a, V):
    """A_{a,S} by scanning every member, plus the member range of prefix a."""
    allowed = {v for v in range(V) if any(_is_prefix(tuple(a) + (v,), s) for s in members)}
    n_with = sum(_is_prefix(a, s) for s in members)
    if n_with == 0:
        return None
    lo = sum(1 for s in members if s < tuple(a))
    return allowed, lo, lo + n_with


def _bits(mask_row, V):
    return {v for v in range(V) if (int(mask_row[v >> 5]) >> (v & 31)) & 1}


def _random_prefix_free_set(rng, V, L_max, n, eos):
    rows = set()
    for _ in range(n):
        if eos:
            ell = int(rng.integers(1, L_max))
            rows.add(tuple(int(x) for x in rng.integers(0, V - 1, size=ell)) + (V - 1,))
        else:
            rows.add(tuple(int(x) for x in rng.integers(0, V, size=L_max)))
    return list(rows)


def test_sorted_table_equals_library_sort_tiny_config():
    w = CONFIGS["tiny"]
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    expect = sorted(set(_rows_of(tok, off)))
    got = _rows_of(*S.rows())
    assert got == expect
    assert S.N == len(expect) == 256 and S.l_max == 3 and S.E == 768


@pytest.mark.parametrize("name,n", [("genret", 5000), ("llm", 20000), ("large", 20000)])
def test_sorted_table_equals_library_sort_scaled(name, n):
    w = scaled(name, n_draws=n)
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    expect = sorted(set(_rows_of(tok, off)))
    assert _rows_of(*S.rows()) == expect
    assert S.N == len(expect)
    assert S.l_max == max(len(r) for r in expect)


def test_duplicates_collapse_and_input_order_is_irrelevant():
    rows = [(3, 1), (0, 2), (3, 1), (0, 1), (3, 0)]
    a = oracle.OracleSet(*_csr(rows), 4)
    b = oracle.OracleSet(*_csr(rows[::-1]), 4)
    assert _rows_of(*a.rows()) == _rows_of(*b.rows()) == [(0, 1), (0, 2), (3, 0), (3, 1)]


@pytest.mark.parametrize("rows,V,code", [
    ([(1, 2), ()], 4, oracle.ERR_EMPTY),
    ([(1, 2), (1, 4)], 4, oracle.ERR_TOKEN),
    ([(1, 2), (-1, 0)], 4, oracle.ERR_TOKEN),
    ([(1, 2), (1, 2, 3)], 4, oracle.ERR_PREFIX),
    ([(1, 2, 3), (1, 2)], 4, oracle.ERR_PREFIX),
    ([], 4, oracle.ERR_EMPTY),
])
def test_build_rejects(rows, V, code):
    with pytest.raises(oracle.OracleError) as e:
        oracle.OracleSet(*_csr(rows), V)
    assert e.value.code == code


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("eos", [False, True])
def test_mask_and_range_brute_force_all_prefixes(seed, eos):
    rng = np.random.default_rng(1000 + seed)
    V = int(rng.integers(2, 9))
    L = int(rng.integers(2, 5))
    members = _random_prefix_free_set(rng, V, L, int(rng.integers(1, 40)), eos)
    S = oracle.OracleSet(*_csr(members), V)
    members = sorted(members)
    # every sequence of length 0..L over the vocabulary, member prefix or not
    for ell in range(L + 1):
        for a in itertools.product(range(V), repeat=ell):
            pref = np.zeros((1, max(L, 1)), np.int32)
            pref[0, :ell] = a
            mask, lo, hi, status = S.mask(pref, [ell])
            bm = _brute_mask(members, a, V)
            if bm is None:
                assert status[0] == 1 and lo[0] == -1 and hi[0] == -1 and not mask.any()
                continue
            allowed, blo, bhi = bm
            assert status[0] == 0
            assert _bits(mask[0], V) == allowed
            assert (int(lo[0]), int(hi[0])) == (blo, bhi)
            # a complete member has an empty valid set and a range of one row
            if tuple(a) in members:
                assert not allowed and bhi - blo == 1
            # partition invariant: children's ranges tile the parent's range
            tot, cursor = 0, blo
            for v in sorted(allowed):
                p2 = pref.copy()
                p2[0, ell] = v if ell < pref.shape[1] else 0
                if ell >= pref.shape[1]:
                    continue
                _, clo, chi, cst = S.mask(p2, [ell + 1])
                assert cst[0] == 0 and clo[0] == cursor
                cursor = int(chi[0])
                tot += int(chi[0] - clo[0])
            if allowed:
                assert tot == bhi - blo and cursor == bhi


@pytest.mark.parametrize("name,n", [("tiny", 256), ("llm", 3000), ("large", 3000)])
def test_mask_matches_lower_bound_characterisation(name, n):
    """Section 3.2: v is valid after prefix a iff a+[v] is a prefix of the first row >= a+[v]."""
    w = scaled(name, n_draws=n)
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    table = _rows_of(*S.rows())
    rng = np.random.default_rng(7)
    for _ in range(25):
        r = table[int(rng.integers(0, len(table)))]
        ell = int(rng.integers(0, len(r)))
        a = r[:ell]
        pref = np.zeros((1, S.l_max), np.int32)
        pref[0, :ell] = a
        mask, lo, hi, status = S.mask(pref, [ell])
        assert status[0] == 0
        got = _bits(mask[0], w.V)
        # check every token of a small vocabulary, a sample (plus all set bits) of a large one
        cand = range(w.V) if w.V <= 64 else set(rng.integers(0, w.V, 300).tolist()) | got
        for v in cand:
            key = a + (v,)
            i = bisect.bisect_left(table, key)
            valid = i < len(table) and _is_prefix(key, table[i])
            assert (v in got) == valid
        assert int(lo[0]) == bisect.bisect_left(table, a)
        assert int(hi[0]) - int(lo[0]) == sum(_is_prefix(a, s) for s in table[int(lo[0]):int(hi[0]) + 1])


def test_full_set_gives_all_ones_and_single_member_gives_one_bit():
    V, L = 5, 3
    full = list(itertools.product(range(V), repeat=L))
    S = oracle.OracleSet(*_csr(full), V)
    for ell in range(L):
        for a in itertools.product(range(V), repeat=ell):
            pref = np.zeros((1, L), np.int32)
            pref[0, :ell] = a
            mask, lo, hi, st = S.mask(pref, [ell])
            assert _bits(mask[0], V) == set(range(V))
            assert int(hi[0] - lo[0]) == V ** (L - ell)
    one = oracle.OracleSet(*_csr([(4, 0, 2)]), V)
    for ell, want in [(0, {4}), (1, {0}), (2, {2}), (3, set())]:
        pref = np.array([[4, 0, 2]], np.int32)
        mask, lo, hi, st = one.mask(pref, [ell])
        assert _bits(mask[0], V) == want and (int(lo[0]), int(hi[0])) == (0, 1)


def test_bits_beyond_vocabulary_are_zero():
    V = 37
    rows = [(v, 0) for v in range(V)]
    S = oracle.OracleSet(*_csr(rows), V)
    mask, *_ = S.mask(np.zeros((1, 2), np.int32), [0])
    assert mask.shape == (1, 2)
    assert int(mask[0, 0]) == 0xFFFFFFFF and int(mask[0, 1]) == (1 << 5) - 1


@pytest.mark.parametrize("eos", [False, True])
def test_verify_candidates_against_a_scan_over_every_member(eos):
    """Algorithm 2, lines 4-6: a candidate t is valid iff a+[t] is a prefix of some member (scan),
    the row index is the number of members smaller than a+[t] (Python tuple order), and the
    extended mask carries exactly the valid candidates."""
    rng = np.random.default_rng(12 + eos)
    V, L = 7, 4
    members = sorted(_random_prefix_free_set(rng, V, L, 60, eos))
    S = oracle.OracleSet(*_csr(members), V)
    prefixes = [p for ell in range(0, L) for p in itertools.product(range(V), repeat=ell)]
    prefixes = [p for p in prefixes if len(p) < 3 or rng.random() < 0.3]
    n, M = len(prefixes), 5
    pre = np.zeros((n, L), np.int32)
    plen = np.array([len(p) for p in prefixes], np.int32)
    for i, p in enumerate(prefixes):
        pre[i, :len(p)] = p
    cand = rng.integers(-1, V + 1, (n, M)).astype(np.int32)      # includes ids outside the vocabulary
    valid, row_index, mask = S.verify(pre, plen, cand)
    for i, p in enumerate(prefixes):
        want_bits = set()
        for m in range(M):
            t = int(cand[i, m])
            vm = tuple(p) + (t,)
            ok = 0 <= t < V and any(_is_prefix(vm, s) for s in members)
            assert valid[i, m] == ok, (p, t)
            assert row_index[i, m] == sum(1 for s in members if s < vm), (p, t)
            if ok:
                want_bits.add(t)
        assert _bits(mask[i], V) == want_bits


def test_verify_with_all_tokens_as_candidates_reproduces_the_exact_mask():
    """With M = |V| (every token a candidate) the verified mask is A_{a,S} itself (Section 3.2,
    "in theory we should set M = |V|")."""
    w = scaled("genret", n_draws=3000)
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    rng = np.random.default_rng(3)
    rows = _rows_of(*S.rows())
    n = 40
    pre = np.zeros((n, S.l_max), np.int32)
    plen = np.zeros(n, np.int32)
    for i in range(n):
        r = rows[int(rng.integers(0, len(rows)))]
        d = int(rng.integers(0, len(r)))
        pre[i, :d] = r[:d]
        plen[i] = d
    cand = np.tile(np.arange(w.V, dtype=np.int32), (n, 1))
    valid, row_index, mask = S.verify(pre, plen, cand)
    m2, lo, hi, st = S.mask(pre, plen)
    assert np.array_equal(mask, m2)
    # the rows the searches land on lie inside the prefix's member range (or right behind it)
    assert np.all((row_index >= lo[:, None]) & (row_index <= hi[:, None]))
    assert np.all(row_index[valid == 1] < hi[:, None].repeat(w.V, 1)[valid == 1])


def test_end_of_keyword_token_for_sets_with_nested_members():
    """Section 2.1: the valid set of x is {v : x+[v] is a prefix of a member}, and the
    end-of-keyword token is valid as well when x itself is a member.  Checked by a scan over the
    members for every sequence over a small vocabulary; members are nested on purpose."""
    rng = np.random.default_rng(8)
    V, EOK, L = 6, 5, 4
    base = {tuple(int(x) for x in rng.integers(0, V - 1, int(rng.integers(1, L + 1)))) for _ in range(40)}
    members = sorted(base | {m[:k] for m in list(base)[:12] for k in range(1, len(m))})
    assert any(a != b and _is_prefix(a, b) for a in members for b in members)
    with pytest.raises(oracle.OracleError):
        oracle.OracleSet(*_csr(members), V)                      # not prefix-free as it stands
    S = oracle.OracleSet(*_csr(members), V, eok=EOK)
    assert S.N == len(members) and S.l_max == max(len(m) for m in members) + 1
    seqs = [p for ell in range(0, L + 1) for p in itertools.product(range(V - 1), repeat=ell)]
    pre = np.zeros((len(seqs), L + 1), np.int32)
    plen = np.array([len(p) for p in seqs], np.int32)
    for i, p in enumerate(seqs):
        pre[i, :len(p)] = p
    mask, lo, hi, st = S.mask(pre, plen)
    mset = set(members)
    for i, x in enumerate(seqs):
        want = {v for v in range(V - 1) if any(_is_prefix(tuple(x) + (v,), s) for s in members)}
        if tuple(x) in mset:
            want.add(EOK)
        if not want:
            assert st[i] == 1
            continue
        assert st[i] == 0 and _bits(mask[i], V) == want, (x, want)
        assert hi[i] - lo[i] == sum(_is_prefix(x, s) for s in members)
    # a member followed by the end-of-keyword token is complete: empty valid set
    for m in members[:10]:
        full = np.zeros((1, L + 1), np.int32)
        full[0, :len(m)] = m
        full[0, len(m)] = EOK
        mk, _, _, s1 = S.mask(full, np.array([len(m) + 1], np.int32))
        assert s1[0] == 0 and not mk.any()
    with pytest.raises(oracle.OracleError):
        oracle.OracleSet(*_csr([(1, EOK, 2)]), V, eok=EOK)        # the closing token inside a member
