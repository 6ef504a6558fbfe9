"""The paper's top-M mode through the C ABI: disc_topm (Algorithm 2, line 3) and disc_step_topm
(Algorithm 1, lines 5-8 with the mask of Algorithm 2, lines 3-6) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_09135_b200 as disc
from gpu_helpers import LockStep, close, logits_to_host
from workloads import make_contexts, make_lm_weights, make_set, scaled
from workloads.standin_lm import StandInLM

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,pad", [(700, 4), (70_001, 0), (4096, 0), (33, 7)])
def test_top_m_selection_is_the_oracles(dtype, V, pad):
    rng = np.random.default_rng(V)
    n = 12
    x = (rng.standard_normal((n, V + pad)) * 2).astype(np.float32)
    x[0] = np.round(x[0], 1)                           # many equal values
    x[1, rng.integers(0, V, max(1, V // 20))] = np.nan
    x[2, :] = 0.25                                     # every logit the same
    x[3, rng.integers(0, V, max(1, V // 10))] = -np.inf
    x[4, rng.integers(0, V, 3)] = np.inf
    x[5] = -np.abs(x[5]) - 1.0                         # all negative
    x[8] = np.sort(x[8])                               # ascending: every logit beats all earlier ones
    x[9] = np.sort(x[9])[::-1]                         # descending
    x[10] = -np.abs(np.round(x[10], 0))                # zeros of both signs on top, many ties below
    x[10, ::3] *= -1.0                                 # (-0.0 * -1 = +0.0, ties across the two zeros)
    x[11] = np.sort(np.round(x[11], 1))                # ascending with runs of equal values
    logits = torch.as_tensor(x).to(dtype).to(DEV)[:, :V] if pad == 0 else torch.as_tensor(x).to(dtype).to(DEV)[:, :V]
    host, dt = logits_to_host(logits)
    host = np.ascontiguousarray(host)
    done = torch.zeros(n, dtype=torch.uint8, device=DEV)
    done[7] = 1
    for M in (1, 5, 50, 1000, 1024, 1025, V, V + 3):
        cand, lse = disc.disc_topm(logits, V, M, inv_temperature=0.7, done=done, want_lse=True)
        torch.cuda.synchronize()
        want = oracle.topm(host, dt, V, M)
        got = cand.cpu().numpy()
        live = np.arange(n) != 7
        assert np.array_equal(got[live], want[live]), M
        assert np.all(got[7] == -1)
    # the by-product: log-sum-exp over the whole row
    from scipy.special import logsumexp
    z = (host.astype(np.float64) if dt == oracle.F32 else (host.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    z = z * np.float64(np.float32(0.7))
    m, s = lse.cpu().numpy()[:, 0].astype(np.float64), lse.cpu().numpy()[:, 1].astype(np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        got_lse = (m + np.log2(s)) * np.log(2.0)
    for i in (0, 2, 3, 5, 6, 8, 9, 10, 11):
        assert close(got_lse[i], logsumexp(z[i])).all(), i
    assert not np.isfinite(got_lse[1]) and not np.isfinite(got_lse[4])      # NaN / +Inf rows are not finite


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_top_m_sum_survives_a_low_temperature(dtype):
    """The one-pass sum is taken against the first logits a thread sees; with 1/T = 60 a row that
    rises by a few units overflows it, and the plain two-pass sum has to take over."""
    from scipy.special import logsumexp
    rng = np.random.default_rng(11)
    V, n = 50_000, 6
    x = (rng.standard_normal((n, V)) * 3).astype(np.float32)
    x[0] = np.sort(x[0])
    x[1] = np.sort(x[1])[::-1]
    x[2] = -300.0
    x[3, :] = -np.inf
    logits = torch.as_tensor(x).to(dtype).to(DEV)
    host, dt = logits_to_host(logits)
    cand, lse = disc.disc_topm(logits, V, 50, inv_temperature=60.0, want_lse=True)
    torch.cuda.synchronize()
    assert np.array_equal(cand.cpu().numpy(), oracle.topm(np.ascontiguousarray(host), dt, V, 50))
    z = (host.astype(np.float64) if dt == oracle.F32 else (host.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    z = z * np.float64(np.float32(60.0))
    m, s = lse.cpu().numpy()[:, 0].astype(np.float64), lse.cpu().numpy()[:, 1].astype(np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        got = (m + np.log2(s)) * np.log(2.0)
    for i in (0, 1, 2, 4, 5):
        assert close(got[i], logsumexp(z[i])).all(), i
    assert got[3] == -np.inf


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_top_m_when_the_sample_misleads(dtype):
    """The one-pass selection takes its threshold from 8,192 logits in evenly spaced runs of 256
    bytes.  Rows whose largest logits sit exactly there make that threshold too high: with 15 of
    them there the second, lower threshold has to succeed, with 1,500 there only the histogram
    passes can."""
    V, n, M = 128_256, 4, 50
    epv = 4 if dtype == torch.float32 else 8
    nvec, runs = V // epv, 8192 // epv // 16
    sampled = np.concatenate([np.arange((c * nvec) // runs * epv, ((c * nvec) // runs + 16) * epv) for c in range(runs)])
    rng = np.random.default_rng(5)
    x = rng.standard_normal((n, V)).astype(np.float32)
    order = np.argsort(-x, axis=1)
    for i, n_top in enumerate((15, 1500, 0, 40)):
        # the n_top largest values of the row go to sampled places, swapped with what was there
        dst = rng.choice(sampled, n_top, replace=False)
        src = order[i, :n_top]
        keep = x[i, dst].copy()
        x[i, dst] = x[i, src]
        x[i, src] = keep
    logits = torch.as_tensor(x).to(dtype).to(DEV)
    host, dt = logits_to_host(logits)
    for M in (50, 1000):
        cand, lse = disc.disc_topm(logits, V, M, want_lse=True)
        torch.cuda.synchronize()
        assert np.array_equal(cand.cpu().numpy(), oracle.topm(np.ascontiguousarray(host), dt, V, M)), M
    from scipy.special import logsumexp
    z = (host.astype(np.float64) if dt == oracle.F32 else (host.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    m, sv = lse.cpu().numpy()[:, 0].astype(np.float64), lse.cpu().numpy()[:, 1].astype(np.float64)
    assert close((m + np.log2(sv)) * np.log(2.0), logsumexp(z, axis=1)).all()


def test_top_m_selection_fuzz():
    """Random shapes, alignments, value distributions and M against the oracle's ordering."""
    rng = np.random.default_rng(2024)
    for case in range(48):
        V = int(rng.choice([1, 2, 7, 8, 9, 255, 256, 257, 1023, 1024, 1025, 2048, 8191, 8192, 8193, 20_000, 33_333]))
        if case % 3 == 0:
            V = int(rng.integers(1, 40_000))
        n = int(rng.integers(1, 6))
        pad = int(rng.integers(0, 9))
        dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
        kind = case % 6
        x = rng.standard_normal((n, V + pad)).astype(np.float32) * float(rng.choice([0.01, 1.0, 30.0]))
        if kind == 1:
            x = np.round(x)                              # few distinct values: long runs of ties
        elif kind == 2:
            x = rng.standard_cauchy((n, V + pad)).astype(np.float32)
        elif kind == 3:
            x[:] = float(rng.standard_normal())          # one value everywhere
        elif kind == 4:
            x[rng.random(x.shape) < 0.05] = np.nan
            x[rng.random(x.shape) < 0.05] = -np.inf
        elif kind == 5:
            x = np.sort(x, axis=1) if rng.random() < 0.5 else -np.sort(-x, axis=1)
        logits = torch.as_tensor(x).to(dtype).to(DEV)[:, :V]
        host, dt = logits_to_host(logits)
        host = np.ascontiguousarray(host)
        for M in {1, int(rng.integers(1, 1025)), min(V, 1024), int(rng.integers(1, 3000))}:
            cand = disc.disc_topm(logits, V, M)
            torch.cuda.synchronize()
            assert np.array_equal(cand.cpu().numpy(), oracle.topm(host, dt, V, M)), (case, V, pad, dtype, kind, M)


CASES = [("llm", dict(n_draws=200_000, B=8, K=16, d=64), 50, 1.0),
         ("llm", dict(n_draws=50_000, B=4, K=8, d=64, V=32_003), 7, 0.8),
         ("large", dict(n_draws=300_000, B=8, K=16, d=64), 100, 1.0),
         ("genret", dict(B=32, K=8), 16, 1.0),
         ("tiny", {}, 5, 1.0)]


@pytest.mark.parametrize("name,over,M,inv_t", CASES)
def test_top_m_decode_in_lockstep_with_the_oracle(name, over, M, inv_t):
    w = scaled(name, **over)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    S = oracle.OracleSet(tok, off, w.V)
    try:
        lm = StandInLM(*make_lm_weights(w), w.logits, DEV)
        ctx = torch.as_tensor(make_contexts(w), device=DEV)
        ls = LockStep(G, S, w.R, with_mask=(w.V <= 40_000))
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        seed = 5 + w.index
        for t in range(G.l_max):
            logits = lm.logits(prev)

            def run(state, seq, out):
                disc.disc_step_topm(G, logits, state, M, seq, inv_temperature=inv_t, seed=seed, step=t, out=out)
                return logits

            def ostep(hl, dt, pre, depth, done, **kw):
                return S.step_topm(hl, dt, M, pre, depth, done, **kw)

            # the mask output of the top-M mode is the mask of the verified candidates, not the
            # exact valid set LockStep compares with: checked separately below
            keep_mask = ls.out.mask
            ls.out.mask = None
            ls.step(None, t, seed, inv_t, run=run, oracle_step=ostep)
            ls.out.mask = keep_mask
            prev = torch.where(ls.out.token >= 0, ls.out.token.to(torch.int64), prev)
        assert bool(ls.state.done.all())
        print(f"[top-{M} {name}] rows*steps checked={ls.checked} dead ends={ls.stuck} near-ties={ls.near_ties} "
              f"max rel logw err={ls.max_err:.2e}")
        assert ls.near_ties <= max(2, ls.checked // 1000)
    finally:
        G.close()
        S.close()


def test_with_every_token_a_candidate_the_step_is_disc_step():
    w = scaled("llm", n_draws=20_000, V=1000, B=8, K=8, d=64)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        lm = StandInLM(*make_lm_weights(w), "bf16", DEV)
        ctx = torch.as_tensor(make_contexts(w), device=DEV)
        sa = disc.disc_state_init(G, w.R, device=DEV)
        sb = sa.clone()
        seq_a = torch.full((w.R, G.l_max), -1, dtype=torch.int32, device=DEV)
        seq_b = seq_a.clone()
        oa = disc.StepOutputs.empty(w.R, DEV, mask_words=G.W)
        ob = disc.StepOutputs.empty(w.R, DEV, mask_words=G.W)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        for t in range(G.l_max):
            logits = lm.logits(prev)
            disc.disc_step(G, logits, sa, seed=9, step=t, seq_tokens=seq_a, out=oa)
            disc.disc_step_topm(G, logits, sb, w.V, seq_b, seed=9, step=t, out=ob)
            torch.cuda.synchronize()
            assert torch.equal(oa.token, ob.token) and torch.equal(oa.status, ob.status)
            assert torch.equal(oa.mask, ob.mask)
            for k in ("node", "lo", "hi", "depth", "done"):
                assert torch.equal(getattr(sa, k), getattr(sb, k)), k
            assert torch.allclose(sa.logw, sb.logw, rtol=0, atol=2e-5)
            prev = torch.where(oa.token >= 0, oa.token.to(torch.int64), prev)
        assert bool(sa.done.all())
    finally:
        G.close()


def test_top_m_mask_is_the_verified_candidates():
    w = scaled("llm", n_draws=100_000, B=8, K=8, d=64)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    S = oracle.OracleSet(tok, off, w.V)
    try:
        lm = StandInLM(*make_lm_weights(w), "bf16", DEV)
        ctx = torch.as_tensor(make_contexts(w), device=DEV)
        st = disc.disc_state_init(G, w.R, device=DEV)
        seq = torch.full((w.R, G.l_max), -1, dtype=torch.int32, device=DEV)
        out = disc.StepOutputs.empty(w.R, DEV, mask_words=G.W)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        M = 200
        for t in range(3):
            logits = lm.logits(prev)
            seq_before = seq.cpu().numpy()
            depth = st.depth.cpu().numpy().copy()
            live = st.done.cpu().numpy() == 0
            _, cand = disc.disc_step_topm(G, logits, st, M, seq, seed=2, step=t, out=out)
            torch.cuda.synchronize()
            valid, _, want_mask = S.verify(seq_before, depth, cand.cpu().numpy())
            got = out.mask.cpu().numpy().view(np.uint32)
            has = valid.any(axis=1)
            assert np.array_equal(got[live & has], want_mask[live & has])
            prev = torch.where(out.token >= 0, out.token.to(torch.int64), prev)
    finally:
        G.close()
        S.close()
