"""Pins for the oracle's top-M mode (Algorithm 2, lines 3-6 inside Algorithm 1, lines 5-8).

What fixes the expected values: numpy's lexsort for the M largest logits (value descending, then
token id ascending, NaN last); the brute-force valid set (a scan over every member) intersected with
that selection, and scipy's fp64 logsumexp over it, for the mask and the probability mass; the
special case M = |V|, where the top-M step must equal the exact-mask step in every output; and the
dead end (no candidate valid), which the paper's Algorithm 1 rejects by its test "a in S"."""
import numpy as np
import pytest
from scipy.special import logsumexp

import oracle
from helpers import bf16_bits_to_f64, csr, f32_to_bf16_bits, rows_of, valid_set
from workloads import make_set, scaled


def _numpy_topm(z, M):
    key = np.where(np.isnan(z), -np.inf, z)
    order = np.lexsort((np.arange(z.shape[0]), -key, np.isnan(z)))      # last key is the primary one
    return np.sort(order[:M])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_top_m_selection_matches_numpy_with_ties_and_nan(dtype):
    rng = np.random.default_rng(4)
    V, n = 700, 30
    x = np.round(rng.standard_normal((n, V)) * 2, 1).astype(np.float32)      # many equal values
    x[3, rng.integers(0, V, 40)] = np.nan
    x[4, :] = 1.5                                                             # every logit the same
    x[5, rng.integers(0, V, 50)] = -np.inf
    x[6, rng.integers(0, V, 5)] = np.inf
    if dtype == "bf16":
        raw = f32_to_bf16_bits(x)
        z = bf16_bits_to_f64(raw)
        args = (raw, oracle.BF16)
    else:
        z = x.astype(np.float64)
        args = (x, oracle.F32)
    for M in (1, 7, 50, 699, 700):
        got = oracle.topm(*args, V, M)
        for i in range(n):
            assert np.array_equal(got[i], _numpy_topm(z[i], M)), (M, i)
    assert np.array_equal(oracle.topm(*args, V, 4)[4], [0, 1, 2, 3])          # ties go to the lower id


def _world():
    w = scaled("llm", n_draws=3000, V=400)
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    table = rows_of(*S.rows())
    rng = np.random.default_rng(9)
    n = 48
    prefix = np.zeros((n, S.l_max), np.int32)
    depth = np.zeros(n, np.int32)
    for i in range(n):
        r = table[int(rng.integers(0, len(table)))]
        depth[i] = int(rng.integers(0, len(r)))
        prefix[i, :depth[i]] = r[:depth[i]]
    depth[:6] = 0                                                             # some rows at the empty prefix
    x = (rng.standard_normal((n, w.V)) * 2).astype(np.float32)
    return w, S, table, prefix, depth, x


def test_with_every_token_a_candidate_the_step_is_the_exact_mask_step():
    w, S, table, prefix, depth, x = _world()
    a = S.step(x, oracle.F32, prefix, depth, seed=12, step=3, inv_temperature=0.9)
    b = S.step_topm(x, oracle.F32, w.V, prefix, depth, seed=12, step=3, inv_temperature=0.9)
    for k in a:
        assert np.array_equal(a[k], b[k], equal_nan=True), k


@pytest.mark.parametrize("M", [1, 5, 50])
def test_mask_and_mass_are_those_of_the_valid_tokens_among_the_m_most_probable(M):
    w, S, table, prefix, depth, x = _world()
    o = S.step_topm(x, oracle.F32, M, prefix, depth, seed=2, step=1)
    z = x.astype(np.float64)
    dead = 0
    for i in range(prefix.shape[0]):
        A = set(valid_set(table, prefix[i, :depth[i]], w.V))
        cand = _numpy_topm(z[i], M)
        ok = sorted(A & set(cand.tolist()))
        assert o["n_children"][i] == len(ok)
        np.testing.assert_allclose(o["lse_all"][i], logsumexp(z[i]), atol=1e-12)
        if not ok:
            dead += 1
            assert o["status"][i] == 1 and o["token"][i] == -1 and o["done"][i] == 1 and o["log_mass"][i] == -np.inf
            continue
        assert o["status"][i] == 0 and o["token"][i] in ok
        np.testing.assert_allclose(o["lse_ok"][i], logsumexp(z[i, ok]), atol=1e-12)
        np.testing.assert_allclose(o["log_mass"][i], logsumexp(z[i, ok]) - logsumexp(z[i]), atol=1e-12)
        np.testing.assert_allclose(o["logq"][i], z[i, o["token"][i]] - logsumexp(z[i, ok]), atol=1e-12)
        # the mass can only shrink against the exact mask (M = |V|)
        assert o["lse_ok"][i] <= logsumexp(z[i, sorted(A)]) + 1e-12
        # cursor: range of the extended prefix
        p2 = prefix[i].copy()
        p2[depth[i]] = o["token"][i]
        _, lo2, hi2, _ = S.mask(p2[None, :], [depth[i] + 1])
        assert (o["lo"][i], o["hi"][i]) == (lo2[0], hi2[0])
    if M == 1:
        assert dead > 0            # with one candidate most rows must run into a dead end


def test_top_m_draws_follow_the_restricted_distribution():
    """Token frequencies over many rows with the same logits follow softmax over the valid
    candidates (chi-square)."""
    from scipy.stats import chisquare
    V = 64
    members = [(v,) for v in range(0, V, 3)]
    S = oracle.OracleSet(*csr(members), V)
    rng = np.random.default_rng(0)
    z = (rng.standard_normal(V) * 1.5).astype(np.float32)
    M = 20
    cand = _numpy_topm(z.astype(np.float64), M)
    ok = sorted(set(cand.tolist()) & {m[0] for m in members})
    assert 3 <= len(ok) < len(members)
    n = 100_000
    o = S.step_topm(np.tile(z, (n, 1)), oracle.F32, M, np.zeros((n, 1), np.int32), np.zeros(n, np.int32),
                    seed=31, step=0, n_threads=8)
    p = np.exp(z[ok].astype(np.float64) - logsumexp(z[ok].astype(np.float64)))
    counts = np.array([(o["token"] == v).sum() for v in ok])
    assert counts.sum() == n
    assert chisquare(counts, p * n).pvalue > 1e-3
