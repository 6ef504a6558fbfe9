"""disc_project_step: the last projection fused with the decoding step, through the C ABI.

What is checked: (1) the logits the tensor-core projection produces against an fp64 product of the
same bf16 inputs, within one bf16 rounding; (2) every step of a decode in lock-step with the oracle,
which is handed the logits the kernel produced (store_all) and the state the GPU started from;
(3) that writing only the pieces of the logits the step reads changes no result, bit for bit, and
leaves the rest of the buffer alone; (4) argument checks."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_09135_b200 as disc
from gpu_helpers import LockStep
from workloads import make_contexts, make_lm_weights, make_set, scaled
from workloads.standin_lm import StandInLM

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _padded(R, V, fill=float("nan")):
    Vp = (V + 7) // 8 * 8            # 16-byte row pitch
    return torch.full((R, Vp), fill, dtype=torch.bfloat16, device=DEV)[:, :V]


@pytest.mark.parametrize("R,V,d", [(128, 4096, 256), (208, 32003, 1024), (130, 1000, 72), (1, 300, 8)])
def test_projection_logits_within_one_bf16_rounding_of_the_exact_product(R, V, d):
    w = scaled("llm", V=V, n_draws=5000, B=1, K=1, d=d)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        g = torch.Generator().manual_seed(R * 7 + d)
        h = torch.randn(R, d, generator=g).to(torch.bfloat16)
        wt = (torch.randn(V, d, generator=g) / d ** 0.5).to(torch.bfloat16)
        exact = h.double() @ wt.double().T
        state = disc.disc_state_init(G, R, device=DEV)
        logits = _padded(R, V)
        scratch = disc.disc_project_scratch(G, R, DEV)
        disc.disc_project_step(G, h.to(DEV), wt.to(DEV), state, logits, scratch, seed=1, step=0, store_all=True)
        disc.disc_project_check(scratch)
        got = logits.double().cpu()
        assert not torch.isnan(got).any()
        # fp32 accumulation of d products, then one rounding to bf16 (relative 2^-9), with slack
        # for a value that sits on a rounding boundary
        tol = exact.abs() * 2.0 ** -8 + 1e-6 * d ** 0.5 + 1e-30
        assert bool(((got - exact).abs() <= tol).all())
        assert float((logits.cpu() == exact.float().to(torch.bfloat16)).float().mean()) > 0.99
    finally:
        G.close()


CASES = [("llm", dict(n_draws=200_000, B=8, K=16, d=64), 1.0),
         ("llm", dict(n_draws=50_000, B=4, K=8, d=72, V=32_003), 0.8),
         ("large", dict(n_draws=300_000, B=9, K=16, d=128), 1.0),
         ("genret", dict(B=40, K=8, d=64), 1.0)]


@pytest.mark.parametrize("name,over,inv_t", CASES)
def test_fused_decode_in_lockstep_with_the_oracle(name, over, inv_t):
    w = scaled(name, **over)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    S = oracle.OracleSet(tok, off, w.V)
    try:
        lm = StandInLM(*make_lm_weights(w), "bf16", DEV)
        wt = lm.projection_rows()
        ctx = torch.as_tensor(make_contexts(w), device=DEV)
        ls = LockStep(G, S, w.R)
        scratch = disc.disc_project_scratch(G, w.R, DEV)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        seed = 77 + w.index
        for t in range(G.l_max):
            h = lm.hidden(prev)
            logits = _padded(w.R, w.V)

            def run(state, seq, out):
                disc.disc_project_step(G, h, wt, state, logits, scratch, inv_temperature=inv_t, seed=seed, step=t,
                                       seq_tokens=seq, out=out, store_all=True)
                disc.disc_project_check(scratch)
                return logits

            ls.step(None, t, seed, inv_t, run=run)
            prev = torch.where(ls.out.token >= 0, ls.out.token.to(torch.int64), prev)
        assert bool(ls.state.done.all())
        print(f"[fused {name}] rows*steps checked={ls.checked} near-ties={ls.near_ties} max rel logw err={ls.max_err:.2e}")
        assert ls.near_ties <= max(2, ls.checked // 1000)
    finally:
        G.close()
        S.close()


@pytest.mark.parametrize("name,over", [("llm", dict(n_draws=200_000, B=16, K=16, d=256)),
                                       ("large", dict(n_draws=300_000, B=16, K=16, d=64))])
def test_writing_only_the_pieces_the_step_reads_changes_nothing(name, over):
    w = scaled(name, **over)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        lm = StandInLM(*make_lm_weights(w), "bf16", DEV)
        wt = lm.projection_rows()
        ctx = torch.as_tensor(make_contexts(w), device=DEV)
        sa = disc.disc_state_init(G, w.R, device=DEV)
        sb = sa.clone()
        su = sa.clone()
        scratch = disc.disc_project_scratch(G, w.R, DEV)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        written = []
        for t in range(G.l_max):
            h = lm.hidden(prev)
            la, lb = _padded(w.R, w.V), _padded(w.R, w.V)
            live = int((sa.done == 0).sum())
            oa = disc.disc_project_step(G, h, wt, sa, la, scratch, seed=5, step=t, store_all=True)
            ob = disc.disc_project_step(G, h, wt, sb, lb, scratch, seed=5, step=t, store_all=False)
            disc.disc_project_check(scratch)
            # the unfused pair on the logits the projection produced
            ou = disc.disc_step(G, la, su, seed=5, step=t)
            torch.cuda.synchronize()
            for k in ("token", "status"):
                assert torch.equal(getattr(oa, k), getattr(ob, k)), (t, k)
            for k in ("node", "lo", "hi", "depth", "done"):
                assert torch.equal(getattr(sa, k), getattr(sb, k)), (t, k)
            assert torch.equal(sa.logw.view(torch.int32), sb.logw.view(torch.int32))
            on = oa.token >= 0                    # rows that were complete already get no logq
            assert torch.equal(oa.logq[on].view(torch.int32), ob.logq[on].view(torch.int32))
            # what was written is what the full projection has there; the rest was left alone
            wr = ~torch.isnan(lb)
            assert torch.equal(lb[wr], la[wr])
            written.append(round(float(wr.float().mean()), 4))
            if t >= 2 and live:
                assert float(wr.float().mean()) < 0.2
            # and the unfused step on the same logits lands on the same tokens
            assert torch.equal(oa.token, ou.token)
            assert torch.allclose(sa.logw, su.logw, rtol=0, atol=2e-5)
            su = sa.clone()
            prev = torch.where(oa.token >= 0, oa.token.to(torch.int64), prev)
        assert bool(sa.done.all())
        print(f"[{name}] share of the logits written per position: {written}")
    finally:
        G.close()


def test_fused_step_argument_checks():
    w = scaled("tiny")
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        R, d = 16, 32
        st = disc.disc_state_init(G, R, device=DEV)
        h = torch.zeros((R, d), dtype=torch.bfloat16, device=DEV)
        wt = torch.zeros((w.V, d), dtype=torch.bfloat16, device=DEV)
        lg = torch.zeros((R, w.V), dtype=torch.bfloat16, device=DEV)
        sc = disc.disc_project_scratch(G, R, DEV)
        disc.disc_project_step(G, h, wt, st, lg, sc)                       # fine
        with pytest.raises(disc.DiscError) as e:                           # scratch too small
            disc.disc_project_step(G, h, wt, st, lg, sc[:64])
        assert e.value.code == -1
        with pytest.raises(disc.DiscError) as e:                           # row pitch not a multiple of 16 bytes
            disc.disc_project_step(G, torch.zeros((R, d + 1), dtype=torch.bfloat16, device=DEV)[:, :d],
                                   wt, st, lg, sc)
        assert e.value.code == -7
        with pytest.raises(disc.DiscError) as e:                           # inverse temperature
            disc.disc_project_step(G, h, wt, st, lg, sc, inv_temperature=0.0)
        assert e.value.code == -1
        with pytest.raises(TypeError):
            disc.disc_project_step(G, h.float(), wt, st, lg, sc)
    finally:
        G.close()
