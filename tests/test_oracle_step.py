"""Pins for the oracle's decoding step (Algorithm 1, lines 5-8) and importance score.

What fixes the expected values here:
  * scipy's fp64 logsumexp / log_softmax with -inf at masked positions;
  * the closed form x(a) = prod_i P_L(A_{a<i,S} | a<i) and the identities
    sum_{a in S} P_L(a)/x(a) = 1,  one constrained draw ~ P_L(a)/x(a),
    E[x] = P_L(S)   (Appendix A, proof of Theorem 3.1), by enumeration of S;
  * the numbers printed in Figure 1's caption (tests/golden/fig1_bias_example.txt);
  * the closed forms of the two-token construction in the proof of Theorem 2.1.
"""
import os

import numpy as np
import pytest
from scipy.special import logsumexp
from scipy.stats import chisquare

import oracle
from helpers import (bf16_bits_to_f64, bits, csr, exact_member_tables, f32_to_bf16_bits, rows_of, tv,
                     valid_set)
from workloads import CONFIGS, make_contexts, make_lm_weights, make_set, scaled
from workloads.standin_lm import markov_table

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _tiny():
    w = CONFIGS["tiny"]
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    Z = markov_table(*make_lm_weights(w))
    members = rows_of(*S.rows())
    return w, S, Z, members


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("inv_t", [1.0, 0.7])
def test_log_softmax_quantities_match_scipy(dtype, inv_t):
    w = scaled("llm", n_draws=4000, V=1000)
    tok, off = make_set(w)
    S = oracle.OracleSet(tok, off, w.V)
    table = rows_of(*S.rows())
    rng = np.random.default_rng(3)
    n = 40
    prefix = np.zeros((n, S.l_max), np.int32)
    depth = np.zeros(n, np.int32)
    for i in range(n):
        r = table[int(rng.integers(0, len(table)))]
        depth[i] = int(rng.integers(0, len(r)))
        prefix[i, :depth[i]] = r[:depth[i]]
    x = (rng.standard_normal((n, w.V)) * 3).astype(np.float32)
    if dtype == "bf16":
        raw = f32_to_bf16_bits(x)
        z = bf16_bits_to_f64(raw) * np.float64(np.float32(inv_t))
        o = S.step(raw, oracle.BF16, prefix, depth, inv_temperature=inv_t, seed=5, step=2)
    else:
        z = x.astype(np.float64) * np.float64(np.float32(inv_t))
        o = S.step(x, oracle.F32, prefix, depth, inv_temperature=inv_t, seed=5, step=2)
    mask, lo, hi, st = S.mask(prefix, depth)
    for i in range(n):
        A = sorted(bits(mask[i], w.V))
        assert A == valid_set(table, prefix[i, :depth[i]], w.V)
        assert o["n_children"][i] == len(A)
        lse_all = logsumexp(z[i])
        lse_ok = logsumexp(z[i, A])
        np.testing.assert_allclose(o["lse_all"][i], lse_all, rtol=0, atol=1e-12)
        np.testing.assert_allclose(o["lse_ok"][i], lse_ok, rtol=0, atol=1e-12)
        np.testing.assert_allclose(o["log_mass"][i], lse_ok - lse_all, rtol=0, atol=1e-12)
        t = int(o["token"][i])
        assert t in A
        np.testing.assert_allclose(o["logq"][i], z[i, t] - lse_ok, atol=1e-12)
        np.testing.assert_allclose(o["logp"][i], z[i, t] - lse_all, atol=1e-12)
        # stage 1: the token's group (8 consecutive ids) maximises log(group mass) + Gumbel noise,
        # noise from the published uniform; stage 2: inverse CDF inside that group
        groups = {}
        for v in A:
            groups.setdefault(v >> 3, []).append(v)
        scores = {G: logsumexp(z[i, vs]) - np.log(-np.log(oracle.group_uniform(5, 2, i, G)))
                  for G, vs in groups.items()}
        Gw = max(sorted(scores), key=lambda G: scores[G])
        assert t >> 3 == Gw
        np.testing.assert_allclose(o["best"][i], scores[Gw], atol=1e-12)
        vs = groups[Gw]
        cum = np.cumsum(np.exp(z[i, vs] - z[i, vs].max()))
        target = oracle.ingroup_uniform(5, 2, i, Gw) * cum[-1]
        assert t == vs[min(len(vs) - 1, int(np.searchsorted(cum, target, side="right")))]
        # range of the extended prefix and leaf test
        p2 = prefix[i].copy()
        p2[depth[i]] = t
        _, lo2, hi2, _ = S.mask(p2[None, :], [depth[i] + 1])
        assert (o["lo"][i], o["hi"][i]) == (lo2[0], hi2[0])
        assert bool(o["done"][i]) == (tuple(p2[:depth[i] + 1]) in set(table))
        assert o["status"][i] == 0


def test_sampled_token_frequencies_follow_masked_softmax():
    """Algorithm 1, line 7: t ~ P.mask/|P.mask|_1; chi-square over 200k independent rows."""
    w, S, Z, members = _tiny()
    a = members[17][:1]
    A = valid_set(members, a, w.V)
    assert len(A) >= 3
    n = 200_000
    prefix = np.tile(np.array(a + (0, 0), np.int32), (n, 1))
    logits = np.tile(Z[a[0]], (n, 1))
    o = S.step(logits, oracle.F32, prefix, np.full(n, 1, np.int32), seed=11, step=1, n_threads=8)
    z = Z[a[0]].astype(np.float64)
    p = np.exp(z[A] - logsumexp(z[A]))
    counts = np.array([(o["token"] == v).sum() for v in A])
    assert counts.sum() == n
    assert chisquare(counts, p * n).pvalue > 1e-3


def test_importance_score_closed_form_and_normalisation_identity():
    """x(a) from the oracle's per-step log_mass equals the closed form; sum_a P_L(a)/x(a) = 1."""
    w, S, Z, members = _tiny()
    ctx = int(make_contexts(w)[0])
    logP, logx = exact_member_tables(members, Z, ctx, w.V)
    got = np.zeros(len(members))
    for i in range(3):
        prefix = np.array([m[:i] + (0,) * (3 - i) for m in members], np.int32)
        prev = np.array([ctx if i == 0 else m[i - 1] for m in members])
        o = S.step(Z[prev], oracle.F32, prefix, np.full(len(members), i, np.int32), seed=1, step=i)
        got += o["log_mass"]
    np.testing.assert_allclose(got, logx, atol=1e-10)
    assert abs(np.exp(logP - logx).sum() - 1.0) < 1e-12
    assert np.all(logx <= 1e-12)


def test_single_constrained_draw_distribution_and_mean_score():
    """K = 1: output ~ P_L(a)/x(a) exactly; E[x] = P_L(S) (Appendix A)."""
    w, S, Z, members = _tiny()
    ctx = 9
    logP, logx = exact_member_tables(members, Z, ctx, w.V)
    p_hat = np.exp(logP - logx)
    n = 300_000
    o = S.decode_markov(Z, np.full(n, ctx, np.int32), 1, seed=2024, n_threads=8)
    index = {m: j for j, m in enumerate(members)}
    which = np.array([index[tuple(s)] for s in o["seq"][:, 0, :].tolist()])
    emp = np.bincount(which, minlength=len(members)) / n
    floor = np.sqrt(p_hat * (1 - p_hat) / n).sum() * np.sqrt(2 / np.pi) * 0.5
    assert tv(emp, p_hat) < 1.3 * floor
    # every draw's accumulated score equals the closed form of the member it produced
    np.testing.assert_allclose(o["logw"][:, 0], logx[which], atol=1e-10)
    # mean score -> P_L(S)
    PLS = np.exp(logP).sum()
    x = np.exp(o["logw"][:, 0])
    assert abs(x.mean() - PLS) < 5 * x.std() / np.sqrt(n)
    assert np.all(o["len"] == 3) and np.all(o["idx"] == 0)


def test_figure1_worked_example():
    rows = [l.strip() for l in open(os.path.join(GOLD, "fig1_bias_example.txt")) if l[0] != "#"]
    want = {}
    for l in rows:
        name, pl, pcd, x = [s.strip() for s in l.split("|")]
        want[name] = (float(pl), float(pcd), float(x))
    vocab = {"soccer": 0, "used": 1, "gloves": 2, "shoes": 3, "shirts": 4, "<ctx>": 5}
    V = 6
    P = np.full((V, V), 1e-300)
    P[5, 0], P[5, 1] = 0.6, 0.4
    P[0, 2], P[0, 3] = 0.1, 0.9
    P[1, 0], P[1, 4] = 0.9, 0.1
    for r in (2, 3, 4):
        P[r, :] = 1.0 / V
    Z = np.log(P / P.sum(1, keepdims=True)).astype(np.float32)
    members = [tuple(vocab[t] for t in name.split()) for name in want]
    S = oracle.OracleSet(*csr(members), V)
    n = 200_000
    o = S.decode_markov(Z, np.full(n, 5, np.int32), 1, seed=8, n_threads=8)
    seqs = [tuple(t for t in s if t >= 0) for s in o["seq"][:, 0, :].tolist()]
    for name, (pl, pcd, x) in want.items():
        m = tuple(vocab[t] for t in name.split())
        sel = np.array([s == m for s in seqs])
        # importance score of this member, identical on every draw that produced it
        np.testing.assert_allclose(np.exp(o["logw"][sel, 0]), x, rtol=1e-6)
        assert abs(sel.mean() - pcd) < 5 * np.sqrt(pcd * (1 - pcd) / n)
        assert abs(pl / x - pcd) < 1e-12          # caption numbers are mutually consistent


@pytest.mark.parametrize("p_b,eps", [(0.3, 0.2), (0.9, 0.01)])
def test_theorem_2_1_two_token_construction(p_b, eps):
    """V = {v1, v2}, S = {v1v1, v1v2, v2v1}: x = (1, 1, eps); constrained decoding gives
    ((1-p_b)/2, (1-p_b)/2, p_b); E[x] = 1 - p_b + p_b*eps = P_L(S)."""
    V = 3                                    # token 2 is only the context
    P = np.array([[0.5, 0.5, 0], [eps, 1 - eps, 0], [1 - p_b, p_b, 0]]) + 1e-300
    Z = np.log(P).astype(np.float32)
    members = [(0, 0), (0, 1), (1, 0)]
    S = oracle.OracleSet(*csr(members), V)
    n = 200_000
    o = S.decode_markov(Z, np.full(n, 2, np.int32), 1, seed=4, n_threads=8)
    seqs = o["seq"][:, 0, :]
    want_cd = [(1 - p_b) / 2, (1 - p_b) / 2, p_b]
    want_x = [1.0, 1.0, eps]
    for m, pcd, x in zip(members, want_cd, want_x):
        sel = (seqs[:, 0] == m[0]) & (seqs[:, 1] == m[1])
        assert abs(sel.mean() - pcd) < 5 * np.sqrt(pcd * (1 - pcd) / n)
        np.testing.assert_allclose(np.exp(o["logw"][sel, 0]), x, rtol=2e-6)
    xs = np.exp(o["logw"][:, 0])
    assert abs(xs.mean() - (1 - p_b + p_b * eps)) < 5 * xs.std() / np.sqrt(n) + 1e-6


def test_degenerate_rows():
    w, S, Z, members = _tiny()
    a = members[0]
    A = valid_set(members, a[:2], w.V)
    logits = np.tile(Z[a[1]], (4, 1)).astype(np.float32)
    prefix = np.tile(np.array(a, np.int32), (4, 1))
    depth = np.array([2, 2, 2, 3], np.int32)
    logits[0, A] = -np.inf                    # no allowed mass
    logits[1, 5] = np.nan                     # NaN in the row
    prefix[2, 1] = (a[1] + 1) % w.V           # maybe not a prefix of any member
    o = S.step(logits, oracle.F32, prefix, depth, done=np.array([0, 0, 0, 1], np.uint8), seed=3)
    assert o["status"][0] & 2 and o["token"][0] == A[0] and o["log_mass"][0] == -np.inf
    assert o["status"][1] & 4 and np.isnan(o["lse_all"][1])
    if not valid_set(members, tuple(prefix[2, :2]), w.V):
        assert o["status"][2] == 1 and o["token"][2] == -1
    assert o["status"][3] == 8 and o["token"][3] == -1
