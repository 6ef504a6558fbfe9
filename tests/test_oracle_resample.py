"""Pins for the oracle's K-way importance draw (Algorithm 1, line 22), the accept test
(Algorithm 1, line 16) and DISC's asymptotic unbiasedness (Theorem 3.1).

Expected values come from: the definition of the draw (probability x_k / sum x_j), scipy's
logsumexp, the exact output law for K = 2 obtained by enumerating S x S (Appendix A:
Q(a) = K * P^(a) * W(a)), the bound KL(P_S || Q) <= sqrt(p_b/(K(1-p_b))) + p_b/(2K(1-p_b)) with
Pinsker's inequality, and E[k] = (1-p_b^K)/(1-p_b) + K p_b^K.
"""
import numpy as np
import pytest
from scipy.special import logsumexp
from scipy.stats import chisquare

import oracle
from helpers import csr, exact_member_tables, rows_of, tv
from workloads import CONFIGS, make_lm_weights, make_set
from workloads.standin_lm import markov_table


def test_k1_always_picks_the_only_candidate():
    lw = np.random.default_rng(0).standard_normal((500, 1)).astype(np.float32) - 3
    o = oracle.resample(lw, seed=3)
    assert np.all(o["idx"] == 0) and np.all(o["status"] == 0)
    np.testing.assert_allclose(o["logz"], lw[:, 0].astype(np.float64), atol=1e-12)


def test_uniform_is_inside_unit_interval_and_fp32_exact():
    u = np.array([oracle.resample_uniform(77, q) for q in range(2000)])
    assert u.min() > 0 and u.max() < 1
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    assert abs(u.mean() - 0.5) < 0.03


@pytest.mark.parametrize("K", [2, 7, 32, 100])
def test_draw_follows_weights(K):
    rng = np.random.default_rng(K)
    lw1 = (rng.standard_normal(K) * 2 - 5).astype(np.float32)
    B = 120_000
    o = oracle.resample(np.tile(lw1, (B, 1)), seed=19)
    p = np.exp(lw1.astype(np.float64) - logsumexp(lw1.astype(np.float64)))
    counts = np.bincount(o["idx"], minlength=K)
    keep = p * B > 5
    assert chisquare(np.append(counts[keep], counts[~keep].sum() + 1e-9),
                     np.append(p[keep], p[~keep].sum() + 1e-9 / B) * B).pvalue > 1e-3
    np.testing.assert_allclose(o["logz"], logsumexp(lw1.astype(np.float64)) - np.log(K), atol=1e-12)
    # the pick is the inverse CDF at the published uniform
    C = np.cumsum(np.exp(lw1.astype(np.float64) - lw1.max()))
    for b in range(0, 2000):
        u = oracle.resample_uniform(19, b)
        assert o["idx"][b] == min(K - 1, int(np.searchsorted(C, u * C[-1], side="right")))


def test_equal_weights_are_uniform_and_offsets_do_not_matter():
    B, K = 90_000, 6
    a = oracle.resample(np.full((B, K), -2.5, np.float32), seed=5)
    b = oracle.resample(np.full((B, K), -80.0, np.float32), seed=5)
    assert np.array_equal(a["idx"], b["idx"])
    assert chisquare(np.bincount(a["idx"], minlength=K)).pvalue > 1e-3


def test_degenerate_weights():
    lw = np.full((3, 4), -np.inf, np.float32)
    lw[1, 2] = -1.0
    lw[2, :] = [np.nan, -1.0, -np.inf, np.nan]
    o = oracle.resample(lw, seed=1)
    u0 = oracle.resample_uniform(1, 0)
    assert o["status"][0] == 2 and o["idx"][0] == int(u0 * 4) and o["logz"][0] == -np.inf
    assert o["status"][1] == 0 and o["idx"][1] == 2
    assert o["status"][2] == 4 and o["idx"][2] == 1


def _small_world(seed=0, V=8, L=3, n_members=120, sharp=1.5):
    rng = np.random.default_rng(seed)
    members = sorted({tuple(int(x) for x in rng.integers(0, V, L)) for _ in range(n_members)})
    Z = (rng.standard_normal((V + 1, V + 1)) * sharp).astype(np.float32)
    Z[:, V] = -1e30                         # the context token is never produced
    return V + 1, members, Z, V             # vocabulary incl. context token id V


def _exact(members, Z, ctx, V):
    logP, logx = exact_member_tables(members, Z, ctx, V)
    P_hat = np.exp(logP - logx)
    PLS = np.exp(logP).sum()
    P_S = np.exp(logP) / PLS
    return logP, logx, P_hat, P_S, PLS


def _empirical(S, members, Z, ctx, K, n, seed):
    o = S.decode_markov(Z, np.full(n, ctx, np.int32), K, seed=seed, n_threads=8)
    index = {m: j for j, m in enumerate(members)}
    pick = o["seq"][np.arange(n), o["idx"], :]
    which = np.array([index[tuple(s)] for s in pick.tolist()])
    return np.bincount(which, minlength=len(members)) / n, o


def test_exact_output_law_for_k2_on_tiny_config():
    w = CONFIGS["tiny"]
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    members = rows_of(*S.rows())
    Z = markov_table(*make_lm_weights(w))
    ctx = 21
    logP, logx, P_hat, P_S, PLS = _exact(members, Z, ctx, w.V)
    x = np.exp(logx)
    Wwin = (P_hat[None, :] * (x[:, None] / (x[:, None] + x[None, :]))).sum(1)
    Q2 = 2 * P_hat * Wwin
    assert abs(Q2.sum() - 1) < 1e-12
    n = 250_000
    emp, _ = _empirical(S, members, Z, ctx, 2, n, seed=31)
    floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(Q2 * (1 - Q2) / n).sum()
    assert tv(emp, Q2) < 1.3 * floor
    assert tv(emp, P_hat) > 2 * floor or tv(Q2, P_hat) < floor   # K=2 law differs from K=1 law


def test_tv_to_target_shrinks_with_k_and_respects_the_kl_bound(capsys):
    """Theorem 3.1 / Appendix A: the K-way draw approaches P_S as K grows."""
    V, members, Z, ctx = _small_world()
    S = oracle.OracleSet(*csr(members), V)
    logP, logx, P_hat, P_S, PLS = _exact(members, Z, ctx, V)
    p_b = 1 - PLS
    assert 0.2 < p_b < 0.95
    report = []
    prev = None
    for K, n in [(1, 200_000), (2, 200_000), (4, 200_000), (8, 100_000), (16, 100_000),
                 (64, 60_000), (256, 30_000), (1024, 10_000)]:
        emp, o = _empirical(S, members, Z, ctx, K, n, seed=100 + K)
        d = tv(emp, P_S)
        floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(P_S * (1 - P_S) / n).sum()
        kl_bound = np.sqrt(p_b / (K * (1 - p_b))) + p_b / (2 * K * (1 - p_b))
        report.append((K, n, d, floor, np.sqrt(kl_bound / 2)))
        assert d <= np.sqrt(kl_bound / 2) + 1.5 * floor
        if prev is not None:
            assert d <= prev + 1.5 * floor                     # no increase beyond noise
        prev = d
        # exp(logZ) is an unbiased estimate of P_L(S)
        zhat = np.exp(o["logz"])
        assert abs(zhat.mean() - PLS) < 5 * zhat.std() / np.sqrt(n) + 1e-9
    exact_tv1 = tv(P_hat, P_S)
    assert abs(report[0][2] - exact_tv1) < 1.5 * report[0][3]
    assert report[-1][2] < 0.25 * exact_tv1 + 1.5 * report[-1][3]
    with capsys.disabled():
        print("\n  K      n     TV(P_S, empirical Q_K)   noise floor   sqrt(KL bound/2)   [p_b = %.3f]" % p_b)
        for K, n, d, f, b in report:
            print("%5d %7d %12.4f %21.4f %14.4f" % (K, n, d, f, b))


def test_accept_phase_expected_draws_and_accepted_law():
    """E[k] = (1-p_b^K)/(1-p_b) + K p_b^K (Theorem 3.1); accepted samples ~ P_S (Appendix A)."""
    V, members, Z, ctx = _small_world(seed=5)
    S = oracle.OracleSet(*csr(members), V)
    logP, logx, P_hat, P_S, PLS = _exact(members, Z, ctx, V)
    p_b = 1 - PLS
    K, n = 4, 200_000
    o = S.decode_markov(Z, np.full(n, ctx, np.int32), K, seed=77, n_threads=8)
    first = oracle.accept(o["logw32"], seed=77)
    # candidates decoded: position of the first accepted one, else K plus K fresh ones
    draws = np.where(first >= 0, first + 1, 2 * K)
    want = (1 - p_b ** K) / (1 - p_b) + K * p_b ** K
    assert abs(draws.mean() - want) < 5 * draws.std() / np.sqrt(n)
    assert abs((first < 0).mean() - p_b ** K) < 5 * np.sqrt(p_b ** K / n)
    acc = first >= 0
    index = {m: j for j, m in enumerate(members)}
    pick = o["seq"][np.arange(n)[acc], first[acc], :]
    which = np.array([index[tuple(s)] for s in pick.tolist()])
    emp = np.bincount(which, minlength=len(members)) / acc.sum()
    floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(P_S * (1 - P_S) / acc.sum()).sum()
    assert tv(emp, P_S) < 1.3 * floor
    # strict comparison with the published uniform
    for b in range(200):
        k = first[b]
        for j in range(K if k < 0 else k + 1):
            ok = np.float64(o["logw32"][b, j]) > np.log(oracle.accept_uniform(77, b, j))
            assert ok == (j == k)


def test_accept_then_resample_output_law_is_the_mixture_of_appendix_a():
    """Lines 11-22 of Algorithm 1 as one routine: with K = 2 the output law is
    (1 - p_b^K) P_S + p_b^K Q_K, where Q_2 is known exactly by enumerating S x S; K = 1 reduces to
    (1 - p_b) P_S + p_b P^ (the single fresh candidate)."""
    V, members, Z, ctx = _small_world(seed=9)
    S = oracle.OracleSet(*csr(members), V)
    logP, logx, P_hat, P_S, PLS = _exact(members, Z, ctx, V)
    p_b = 1 - PLS
    x = np.exp(logx)
    Q = {1: P_hat, 2: 2 * P_hat * (P_hat[None, :] * (x[:, None] / (x[:, None] + x[None, :]))).sum(1)}
    index = {m: j for j, m in enumerate(members)}
    n = 200_000
    for K in (1, 2):
        o = S.decode_markov(Z, np.full(n, ctx, np.int32), 2 * K, seed=500 + K, n_threads=8)
        r = oracle.accept_resample(o["logw32"], seed=500 + K)
        # bookkeeping: accepted column, or a fresh one
        acc = r["first"] >= 0
        assert np.array_equal(r["choice"][acc], r["first"][acc])
        assert np.all((r["choice"][~acc] >= K) & (r["choice"][~acc] < 2 * K))
        assert abs((~acc).mean() - p_b ** K) < 5 * np.sqrt(p_b ** K * (1 - p_b ** K) / n)
        pick = o["seq"][np.arange(n), r["choice"], :]
        emp = np.bincount([index[tuple(s)] for s in pick.tolist()], minlength=len(members)) / n
        want = (1 - p_b ** K) * P_S + p_b ** K * Q[K]
        assert abs(want.sum() - 1) < 1e-12
        floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(want * (1 - want) / n).sum()
        assert tv(emp, want) < 1.3 * floor
        # the mixture is closer to the target than the plain K-way draw it falls back to
        assert tv(want, P_S) < tv(Q[K], P_S)


def test_accept_then_resample_special_cases():
    K = 3
    lw = np.full((4, 2 * K), -1.0, np.float32)
    lw[0, :K] = 0.0                    # x = 1 > eps always: the first candidate is accepted
    lw[1, :K] = -np.inf                # x = 0: never accepted, falls back
    lw[1, K:] = [-np.inf, -2.0, -np.inf]    # only one fresh candidate has weight
    lw[2, :K] = [-np.inf, 0.0, 0.0]    # the second is the first acceptable one
    lw[3, :] = -np.inf                 # nothing acceptable, nothing to weigh: uniform fallback, flagged
    r = oracle.accept_resample(lw, seed=3)
    assert r["first"].tolist()[:3] == [0, -1, 1] and r["choice"].tolist()[:3] == [0, K + 1, 1]
    assert r["first"][3] == -1 and K <= r["choice"][3] < 2 * K and r["status"][3] & 2
    assert abs(r["logz"][1] - (-2.0 - np.log(K))) < 1e-12
