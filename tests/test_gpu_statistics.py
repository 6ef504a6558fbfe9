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
