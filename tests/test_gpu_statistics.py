"""DISC through the CUDA path: the empirical law of the K-way draw approaches the constrained
target P_S(a) = P_L(a) / P_L(S) as K grows (Theorem 3.1), on the tiny workload, with the exact
target obtained by enumerating S.  Total-variation distances are printed."""
import numpy as np
import pytest
import torch

import paper_2504_09135_b200 as disc
from helpers import exact_member_tables, rows_of, tv
from workloads import CONFIGS, make_lm_weights, make_set
from workloads.standin_lm import markov_table

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_tv_to_constrained_target_shrinks_with_k(capsys):
    w = CONFIGS["tiny"]
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    members = rows_of(*disc.disc_set_rows(G))
    Z = markov_table(*make_lm_weights(w))
    ctx = 21
    logP, logx = exact_member_tables(members, Z, ctx, w.V)
    P_S = np.exp(logP - np.logaddexp.reduce(logP))
    P_hat = np.exp(logP - logx)
    Zd = torch.as_tensor(Z, device=DEV)
    code = {m: j for j, m in enumerate(members)}
    lut = np.full(w.V ** 3, -1, np.int64)
    for m, j in code.items():
        lut[(m[0] * w.V + m[1]) * w.V + m[2]] = j
    report, prev = [], None
    for K, n in [(1, 400_000), (4, 200_000), (16, 100_000), (64, 40_000), (256, 10_000)]:
        dec = disc.DiscDecoder(G, n, K, DEV, want_logq=False, want_logp=False)
        dec.reset()
        prevtok = torch.full((n * K,), ctx, dtype=torch.int64, device=DEV)
        for t in range(G.l_max):
            o = dec.step(Zd.index_select(0, prevtok), t, seed=1000 + K)
            prevtok = o.token.to(torch.int64)
        r = dec.finish(seed=1000 + K)
        tokens = r["tokens"].cpu().numpy().astype(np.int64)
        which = lut[(tokens[:, 0] * w.V + tokens[:, 1]) * w.V + tokens[:, 2]]
        assert which.min() >= 0                       # only members come out
        emp = np.bincount(which, minlength=len(members)) / n
        d = tv(emp, P_S)
        floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(P_S * (1 - P_S) / n).sum()
        report.append((K, n, d, floor))
        if K == 1:
            assert abs(d - tv(P_hat, P_S)) < 1.5 * floor
            assert tv(emp, P_hat) < 1.3 * 0.5 * np.sqrt(2 / np.pi) * np.sqrt(P_hat * (1 - P_hat) / n).sum()
        if prev is not None:
            assert d <= prev + 1.5 * floor
        prev = d
        # exp(logZ) estimates P_L(S) without bias
        zhat = np.exp(r["logz"].cpu().numpy().astype(np.float64))
        assert abs(zhat.mean() - np.exp(logP).sum()) < 5 * zhat.std() / np.sqrt(n) + 1e-9
        del dec
    assert report[-1][2] < 0.35 * report[0][2]
    with capsys.disabled():
        print("\n  CUDA path, tiny workload:   K        n   TV(P_S, empirical)   noise floor")
        for K, n, d, f in report:
            print("%36d %8d %14.4f %15.4f" % (K, n, d, f))
    G.close()


def test_accept_then_resample_law_through_the_cuda_path():
    """Algorithm 1, lines 11-22 through disc_step + disc_accept_resample on a small world (V = 8,
    120 members of length 3, p_b around one half): the output law is (1 - p_b^K) P_S + p_b^K Q_K
    (Appendix A) with Q_2 known by enumerating S x S, the share of fallbacks is p_b^K, and the mean
    number of candidates used follows E[k] = (1 - p_b^K)/(1 - p_b) + K p_b^K (Theorem 3.1)."""
    from helpers import csr
    rng = np.random.default_rng(5)
    V0, L = 8, 3
    members = sorted({tuple(int(t) for t in rng.integers(0, V0, L)) for _ in range(120)})
    V, ctx = V0 + 1, V0                       # the context token is an extra id that is never produced
    Z = (rng.standard_normal((V, V)) * 1.5).astype(np.float32)
    Z[:, ctx] = -1e30
    G = disc.disc_build_set(*csr(members), V)
    logP, logx = exact_member_tables(members, Z, ctx, V)
    PLS = np.exp(logP).sum()
    p_b = 1 - PLS
    assert 0.2 < p_b < 0.95
    P_S = np.exp(logP) / PLS
    P_hat = np.exp(logP - logx)
    x = np.exp(logx)
    Q = {1: P_hat, 2: 2 * P_hat * (P_hat[None, :] * (x[:, None] / (x[:, None] + x[None, :]))).sum(1)}
    lut = np.full(V ** 3, -1, np.int64)
    for j, m in enumerate(members):
        lut[(m[0] * V + m[1]) * V + m[2]] = j
    Zd = torch.as_tensor(Z, device=DEV)
    for K, n in [(1, 300_000), (2, 200_000)]:
        dec = disc.DiscDecoder(G, n, 2 * K, DEV, want_logq=False, want_logp=False)
        dec.reset()
        prevtok = torch.full((n * 2 * K,), ctx, dtype=torch.int64, device=DEV)
        for t in range(G.l_max):
            o = dec.step(Zd.index_select(0, prevtok), t, seed=77 + K)
            prevtok = o.token.to(torch.int64)
        r = dec.finish_accept_resample(seed=77 + K)
        first = r["first"].cpu().numpy()
        tokens = r["tokens"].cpu().numpy().astype(np.int64)
        which = lut[(tokens[:, 0] * V + tokens[:, 1]) * V + tokens[:, 2]]
        assert which.min() >= 0
        emp = np.bincount(which, minlength=len(members)) / n
        want = (1 - p_b ** K) * P_S + p_b ** K * Q[K]
        floor = 0.5 * np.sqrt(2 / np.pi) * np.sqrt(want * (1 - want) / n).sum()
        assert tv(emp, want) < 1.3 * floor
        assert tv(emp, Q[K]) > 2 * floor                 # and it is not the plain K-way law
        rej = (first < 0).mean()
        assert abs(rej - p_b ** K) < 5 * np.sqrt(p_b ** K * (1 - p_b ** K) / n)
        used = np.where(first >= 0, first + 1, 2 * K)
        want_k = (1 - p_b ** K) / (1 - p_b) + K * p_b ** K
        assert abs(used.mean() - want_k) < 5 * used.std() / np.sqrt(n), (K, p_b, used.mean(), want_k)
        del dec
    G.close()
