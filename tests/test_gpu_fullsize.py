"""Parity at the benchmark's full sizes, in the launch configuration bench.py times:
|S| = 10 M draws (about 10^8 table entries), V = 128,256, 4,096 bf16 rows per disc_step launch, and
the 65,536-prefix mask-only stress.  The oracle checks a sample of rows one by one (it needs about
1.5 ms per row and position); masks and ranges of all prefixes are compared in full."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_09135_b200 as disc
from gpu_helpers import LockStep
from workloads import CONFIGS, make_contexts, make_lm_weights, make_prefixes, make_set, scaled
from workloads.standin_lm import StandInLM

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def large():
    w = CONFIGS["large"]
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    S = oracle.OracleSet(tok, off, w.V)
    yield w, tok, off, G, S
    G.close()
    S.close()


def test_full_table_is_identical(large):
    w, tok, off, G, S = large
    assert (G.N, G.E, G.l_max, G.n_nodes) == (S.N, S.E, S.l_max, S.n_nodes)
    gt, go = disc.disc_set_rows(G)
    st, so = S.rows()
    assert np.array_equal(go, so) and np.array_equal(gt, st)
    print(f"large set: N={G.N} E={G.E} nodes={G.n_nodes} levels={G.level_nodes} "
          f"device={G.device_bytes / 1e6:.0f} MB build={G.build_seconds:.2f}s")


def test_full_size_decode_on_sampled_rows(large):
    w, tok, off, G, S = large
    lw = scaled("large", d=256)                      # same logits law, cheaper stand-in projection
    lm = StandInLM(*make_lm_weights(lw), lw.logits, DEV)
    ctx = torch.as_tensor(make_contexts(w), device=DEV)
    rows = np.arange(5, w.R, 43)                     # 96 of the 4,096 rows
    ls = LockStep(G, S, w.R, rows=rows)
    prev = ctx.to(torch.int64).repeat_interleave(w.K)
    seed = 99
    for t in range(G.l_max):
        logits = lm.logits(prev)
        assert logits.shape == (w.R, w.V) and logits.dtype == torch.bfloat16
        ls.step(logits, t, seed)
        prev = torch.where(ls.out.token >= 0, ls.out.token.to(torch.int64), prev)
    assert bool(ls.state.done.all())
    # properties that hold for every row: members only, finite non-positive log-weights
    seq = ls.seq.cpu().numpy()
    lens = (seq >= 0).sum(1)
    assert lens.min() >= w.len_min and lens.max() <= w.len_max
    assert np.all(seq[np.arange(w.R), lens - 1] == w.V - 1)          # every member ends with EOS
    _, lo, hi, st = S.mask(seq, lens.astype(np.int32))
    assert np.all(st == 0) and np.all(hi - lo == 1)
    assert np.array_equal(ls.state.lo.cpu().numpy(), lo)
    logw = ls.state.logw.cpu().numpy()
    assert np.all(np.isfinite(logw)) and np.all(logw <= 1e-4)
    print(f"full-size decode: checked={ls.checked} near-ties={ls.near_ties} max rel logw err={ls.max_err:.2e}")
    assert ls.near_ties <= 2


def test_full_size_mask_stress(large):
    w, tok, off, G, S = large
    mw = CONFIGS["mask"]
    prefix, plen = make_prefixes(mw, tok, off)
    assert prefix.shape[0] == 65_536
    g = disc.disc_mask(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV))
    torch.cuda.synchronize()
    lo_g, hi_g, st_g = g["lo"].cpu().numpy(), g["hi"].cpu().numpy(), g["status"].cpu().numpy()
    step = 4096
    for a in range(0, prefix.shape[0], step):
        m, lo, hi, st = S.mask(prefix[a:a + step], plen[a:a + step])
        assert np.array_equal(st_g[a:a + step], st)
        assert np.array_equal(lo_g[a:a + step], lo) and np.array_equal(hi_g[a:a + step], hi)
        assert np.array_equal(g["mask"][a:a + step].cpu().numpy().view(np.uint32), m)
    assert np.all(st_g == 0)
