"""DiscDecoder's other two ways to take a step: the paper's top-M mode and the fused projection.
(The kernels themselves are checked step by step against the oracle in test_gpu_topm.py and
test_gpu_project.py; here the decode loops built on them.)"""
import numpy as np
import pytest
import torch

import paper_2504_09135_b200 as disc
from workloads import make_contexts, make_lm_weights, make_set, scaled
from workloads.standin_lm import StandInLM

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _setup(name, **over):
    w = scaled(name, **over)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    E, W, b = make_lm_weights(w)
    lm = StandInLM(E, W, b, w.logits, DEV)
    ctx = torch.as_tensor(make_contexts(w))
    t, o = disc.disc_set_rows(G)
    members = {tuple(t[o[i]:o[i + 1]].tolist()) for i in range(len(o) - 1)}
    return w, G, lm, ctx, members


@pytest.mark.parametrize("name,over", [("tiny", {}), ("genret", dict(B=16, K=8))])
def test_top_m_decoder_with_every_token_a_candidate_is_the_exact_decoder(name, over):
    """With M = |V| every token is a candidate, the verified ones are the valid set, and the whole
    decode - tokens, log-weights, the K-way draw - must be the one disc_step gives."""
    w, G, lm, ctx, _ = _setup(name, **over)
    try:
        exact = disc.DiscDecoder(G, w.B, w.K, DEV)
        topm = disc.DiscDecoder(G, w.B, w.K, DEV, top_m=w.V)
        keep = []
        r0 = {k: v.clone() for k, v in exact.decode(lm, ctx, seed=3, keep_logits=keep).items()}
        r1 = topm.replay(keep, seed=3)
        torch.cuda.synchronize()
        assert torch.equal(exact.seq, topm.seq)
        assert torch.equal(exact.state.done, topm.state.done)
        assert torch.allclose(exact.state.logw, topm.state.logw, rtol=1e-5, atol=1e-4)
        assert torch.equal(r0["idx"], r1["idx"]) and torch.equal(r0["tokens"], r1["tokens"])
    finally:
        G.close()


def test_top_m_decoder_ends_rows_in_members_or_dead_ends():
    w, G, lm, ctx, members = _setup("genret", B=16, K=8)
    try:
        dec = disc.DiscDecoder(G, w.B, w.K, DEV, top_m=128)
        dec.decode(lm, ctx, seed=5)
        torch.cuda.synchronize()
        seq, logw = dec.seq.cpu().numpy(), dec.state.logw.cpu().numpy()
        assert bool(dec.state.done.all())
        n_member = 0
        for i in range(dec.R):
            row = tuple(int(t) for t in seq[i] if t >= 0)
            if np.isfinite(logw[i]):
                assert row in members
                n_member += 1
            else:                                    # a dead end: never picked by the K-way draw
                assert logw[i] == -np.inf and row not in members
        assert 0 < n_member
        idx = dec.res["idx"].cpu().numpy()
        lw = logw.reshape(w.B, w.K)
        for b in range(w.B):
            if np.isfinite(lw[b]).any():
                assert np.isfinite(lw[b, idx[b]])
    finally:
        G.close()


def test_decode_from_hidden_vectors_ends_every_row_in_a_member():
    w, G, lm, ctx, members = _setup("genret", B=16, K=8, d=64)
    try:
        dec = disc.DiscDecoder(G, w.B, w.K, DEV)
        r = dec.decode_hidden(lm, ctx, seed=7)
        disc.disc_project_check(dec._proj[1])
        seq = dec.seq.cpu().numpy()
        assert bool(dec.state.done.all()) and bool(torch.isfinite(dec.state.logw).all())
        for i in range(dec.R):
            assert tuple(int(t) for t in seq[i] if t >= 0) in members
        tokens = r["tokens"].cpu().numpy()
        for b in range(w.B):
            assert tuple(int(t) for t in tokens[b] if t >= 0) in members
        with pytest.raises(ValueError):
            disc.DiscDecoder(G, w.B, w.K, DEV, top_m=4).step_hidden(lm.hidden(ctx.repeat_interleave(w.K)),
                                                                   lm.projection_rows(), 0)
    finally:
        G.close()


def test_top_m_decode_replayed_as_a_graph_gives_the_same_result():
    w, G, lm, ctx, _ = _setup("genret", B=16, K=8)
    try:
        dec = disc.DiscDecoder(G, w.B, w.K, DEV, top_m=128)
        keep = []
        dec.decode(lm, ctx, seed=9, keep_logits=keep)
        torch.cuda.synchronize()
        seq, logw, idx = dec.seq.clone(), dec.state.logw.clone(), dec.res["idx"].clone()
        graph = dec.capture(keep, seed=9)
        dec.seq.fill_(-7)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(dec.seq, seq) and torch.equal(dec.res["idx"], idx)
        assert torch.equal(dec.state.logw, logw)
    finally:
        G.close()
