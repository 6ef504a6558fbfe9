"""Pins for the oracle's two samplers of Algorithm 1, line 7 (t ~ P.mask/|P.mask|_1).

oracle.step_plain is the kernel-independent statement (inverse CDF over the allowed tokens with one
uniform); oracle.step draws in two stages over groups of 8 token ids.  What fixes the expected
values: the exact masked softmax computed with scipy in fp64, against which the empirical token
frequencies of BOTH samplers are put by a chi-square test, on valid sets laid out to stress the
grouping: tokens straddling group boundaries, a vocabulary that is not a multiple of 8 with allowed
tokens in the ragged last group, groups with a single allowed token, a group whose only allowed
token has a -inf logit, and groups with three or more allowed tokens.
"""
import numpy as np
import pytest
from scipy.special import logsumexp
from scipy.stats import chisquare

import oracle
from helpers import csr

V = 61                      # not a multiple of 8: the last group holds ids 56..60

LAYOUTS = {
    "straddle_group_boundaries": [6, 7, 8, 9, 15, 16, 23, 24],
    "ragged_last_group": [0, 55, 56, 58, 60],
    "one_token_groups": [1, 10, 19, 28, 37, 46, 59],
    "three_or_more_in_a_group": [16, 17, 19, 22, 23, 40, 41, 42, 43, 44, 45, 46, 47],
    "only_token_of_a_group_has_no_mass": [3, 9, 10, 33],          # logit of 3 is -inf (see below)
    "everything_allowed": list(range(V)),
    "single_group": [24, 26, 31],
}


def _world(name):
    A = LAYOUTS[name]
    S = oracle.OracleSet(*csr([(v,) for v in A]), V)
    rng = np.random.default_rng(sorted(LAYOUTS).index(name) + 100)
    z = (rng.standard_normal(V) * 2.0).astype(np.float32)
    if name == "only_token_of_a_group_has_no_mass":
        z[3] = -np.inf
    return A, S, z


@pytest.mark.parametrize("name", sorted(LAYOUTS))
@pytest.mark.parametrize("sampler", ["plain", "two_stage"])
def test_sampler_follows_the_exact_masked_softmax(name, sampler):
    A, S, z = _world(name)
    n = 120_000
    logits = np.tile(z, (n, 1))
    prefix = np.zeros((n, 1), np.int32)
    depth = np.zeros(n, np.int32)
    f = S.step_plain if sampler == "plain" else S.step
    o = f(logits, oracle.F32, prefix, depth, seed=77, step=3, n_threads=8)
    z64 = z.astype(np.float64)
    p = np.exp(z64[A] - logsumexp(z64[A]))
    counts = np.array([(o["token"] == v).sum() for v in A])
    assert counts.sum() == n                               # only allowed tokens are ever drawn
    keep = p > 0
    assert np.all(counts[~keep] == 0)                      # a token without mass is never drawn
    assert chisquare(counts[keep], p[keep] * n).pvalue > 1e-3
    assert np.all(o["status"] == 0) and np.all(o["done"] == 1)


@pytest.mark.parametrize("name", sorted(LAYOUTS))
def test_samplers_share_everything_but_the_draw(name):
    A, S, z = _world(name)
    n = 64
    rng = np.random.default_rng(5)
    logits = (np.tile(z, (n, 1)) + rng.standard_normal((n, V)).astype(np.float32)).astype(np.float32)
    prefix = np.zeros((n, 1), np.int32)
    depth = np.zeros(n, np.int32)
    a = S.step(logits, oracle.F32, prefix, depth, seed=1, step=0)
    b = S.step_plain(logits, oracle.F32, prefix, depth, seed=1, step=0)
    for k in ("lse_all", "lse_ok", "log_mass", "status"):
        assert np.array_equal(a[k], b[k]), k
    z64 = logits.astype(np.float64)
    np.testing.assert_allclose(b["lse_ok"], logsumexp(z64[:, A], axis=1), atol=1e-12)
    np.testing.assert_allclose(b["logq"], z64[np.arange(n), b["token"]] - b["lse_ok"], atol=1e-12)
    np.testing.assert_allclose(b["logp"], z64[np.arange(n), b["token"]] - b["lse_all"], atol=1e-12)
    # the plain draw is numpy's inverse CDF of the published uniform
    for i in range(n):
        w = np.exp(z64[i, A] - z64[i, A].max())
        cum = np.cumsum(w)
        u = oracle.plain_uniform(1, 0, i)
        assert b["token"][i] == A[min(len(A) - 1, int(np.searchsorted(cum, u * cum[-1], side="right")))]


def test_plain_sampler_temperature_and_bf16():
    A, S, z = _world("three_or_more_in_a_group")
    import torch
    raw = torch.as_tensor(z).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    zb = (raw.astype(np.uint32) << 16).view(np.float32).astype(np.float64) * np.float64(np.float32(0.6))
    n = 100_000
    o = S.step_plain(np.tile(raw, (n, 1)), oracle.BF16, np.zeros((n, 1), np.int32), np.zeros(n, np.int32),
                     inv_temperature=0.6, seed=9, step=1, n_threads=8)
    p = np.exp(zb[A] - logsumexp(zb[A]))
    counts = np.array([(o["token"] == v).sum() for v in A])
    assert counts.sum() == n and chisquare(counts, p * n).pvalue > 1e-3
    np.testing.assert_allclose(o["lse_ok"], logsumexp(zb[A]), atol=1e-12)


def test_plain_sampler_degenerate_rows():
    A, S, z = _world("one_token_groups")
    logits = np.tile(z, (3, 1))
    logits[0, A] = -np.inf                     # no allowed mass: lowest valid id, status 2
    logits[1, 7] = np.nan                      # NaN outside the valid set: status 4, draw still from A
    o = S.step_plain(logits, oracle.F32, np.zeros((3, 1), np.int32), np.zeros(3, np.int32),
                     done=np.array([0, 0, 1], np.uint8), seed=2)
    assert o["status"][0] & 2 and o["token"][0] == A[0] and o["log_mass"][0] == -np.inf
    assert o["status"][1] & 4 and o["token"][1] in A
    assert o["status"][2] == 8 and o["token"][2] == -1
