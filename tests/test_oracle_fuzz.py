"""Property tests (hypothesis) for the oracle: random small sets, prefixes, candidates and logits
against brute force and library routines.  Complements the fixed-seed pins with many small shapes:
every sequence length from 1, vocabularies that are not a multiple of anything, sets with a single
member, prefixes that are members, prefixes outside the set."""
import numpy as np
from hypothesis import given, settings, strategies as st
from scipy.special import logsumexp

import oracle
from helpers import bits, csr, is_prefix, valid_set


@st.composite
def prefix_free_sets(draw):
    V = draw(st.integers(2, 9))
    L = draw(st.integers(1, 4))
    eos = draw(st.booleans()) and V >= 3
    n = draw(st.integers(1, 25))
    rows = set()
    for _ in range(n):
        if eos:   # variable length, closed by the token V-1
            ell = draw(st.integers(0, L - 1)) if L > 1 else 0
            body = tuple(draw(st.integers(0, V - 2)) for _ in range(ell))
            rows.add(body + (V - 1,))
        else:     # fixed length
            rows.add(tuple(draw(st.integers(0, V - 1)) for _ in range(L)))
    return V, sorted(rows)


@settings(max_examples=120, deadline=None)
@given(prefix_free_sets(), st.data())
def test_mask_range_and_verification_against_a_scan(vs, data):
    V, members = vs
    S = oracle.OracleSet(*csr(members), V)
    assert S.N == len(members)
    ell = data.draw(st.integers(0, S.l_max))
    a = tuple(data.draw(st.integers(0, V - 1)) for _ in range(ell))
    if data.draw(st.booleans()) and members:           # bias towards real prefixes
        m = members[data.draw(st.integers(0, len(members) - 1))]
        a = m[:data.draw(st.integers(0, len(m)))]
    pre = np.zeros((1, max(1, S.l_max)), np.int32)
    pre[0, :len(a)] = a
    mask, lo, hi, status = S.mask(pre, [len(a)])
    with_a = [s for s in members if is_prefix(a, s)]
    if not with_a:
        assert status[0] == 1 and not mask.any() and lo[0] == hi[0] == -1
    else:
        assert status[0] == 0
        assert sorted(bits(mask[0], V)) == valid_set(members, a, V)
        assert (lo[0], hi[0]) == (sum(1 for s in members if s < a and not is_prefix(a, s)),
                                  sum(1 for s in members if s < a and not is_prefix(a, s)) + len(with_a))
    # Algorithm 2 on the same prefix with every token (and two ids outside the vocabulary) as candidates
    cand = np.arange(-1, V + 1, dtype=np.int32)[None, :]
    valid, rows, vmask = S.verify(pre, [len(a)], cand)
    for j, t in enumerate(cand[0]):
        vm = tuple(a) + (int(t),)
        assert valid[0, j] == (0 <= t < V and any(is_prefix(vm, s) for s in members))
        assert rows[0, j] == sum(1 for s in members if s < vm)
    assert np.array_equal(vmask, mask)


@settings(max_examples=80, deadline=None)
@given(prefix_free_sets(), st.integers(0, 2 ** 31 - 1), st.sampled_from([0.5, 1.0, 2.0]), st.booleans())
def test_step_quantities_against_library_routines(vs, seed, inv_t, use_bf16):
    V, members = vs
    S = oracle.OracleSet(*csr(members), V)
    rng = np.random.default_rng(seed)
    m = members[int(rng.integers(0, len(members)))]
    d = int(rng.integers(0, len(m)))
    a = m[:d]
    pre = np.zeros((1, max(1, S.l_max)), np.int32)
    pre[0, :d] = a
    x = (rng.standard_normal((1, V)) * 3).astype(np.float32)
    if use_bf16:
        from helpers import bf16_bits_to_f64, f32_to_bf16_bits
        raw = f32_to_bf16_bits(x)
        z = bf16_bits_to_f64(raw) * inv_t
        o = S.step(raw, oracle.BF16, pre, [d], inv_temperature=inv_t, seed=seed, step=3)
    else:
        z = x.astype(np.float64) * inv_t
        o = S.step(x, oracle.F32, pre, [d], inv_temperature=inv_t, seed=seed, step=3)
    z = z[0]
    A = valid_set(members, a, V)
    np.testing.assert_allclose(o["lse_all"][0], logsumexp(z), atol=1e-12)
    np.testing.assert_allclose(o["lse_ok"][0], logsumexp(z[A]), atol=1e-12)
    np.testing.assert_allclose(o["log_mass"][0], logsumexp(z[A]) - logsumexp(z), atol=1e-12)
    t = int(o["token"][0])
    assert t in A and o["n_children"][0] == len(A)
    # the two-stage draw, recomputed from the published uniforms
    groups = {}
    for v in A:
        groups.setdefault(v >> 3, []).append(v)
    scores = {G: logsumexp(z[g]) - np.log(-np.log(oracle.group_uniform(seed, 3, 0, G))) for G, g in groups.items()}
    Gw = max(sorted(scores), key=lambda G: scores[G])
    g = groups[Gw]
    cum = np.cumsum(np.exp(z[g] - z[g].max()))
    pick = g[min(len(g) - 1, int(np.searchsorted(cum, oracle.ingroup_uniform(seed, 3, 0, Gw) * cum[-1], side="right")))]
    second = sorted(scores.values())[-2] if len(scores) > 1 else -np.inf
    if scores[Gw] - second > 1e-9:
        assert t >> 3 == Gw
        if o["ingroup_gap"][0] > 1e-9:
            assert t == pick
    np.testing.assert_allclose(o["logq"][0], z[t] - logsumexp(z[A]), atol=1e-12)
    assert bool(o["done"][0]) == (tuple(a) + (t,) in set(members))
