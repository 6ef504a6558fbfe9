"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Bar: sorted table, masks, ranges, completion flags, statuses bit-exact; log-weights, log-probs and
logZ within 1e-5 relative (|a-b| <= 1e-5*max(1,|b|)); sampled tokens equal unless the oracle's
scores of the two picks differ by less than 1e-5 (counted); resampled index equal unless the
threshold lies within 1e-5 of an interval boundary (counted).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_09135_b200 as disc
from gpu_helpers import TOL, LockStep, assert_near_ties, close, logits_to_host
from helpers import csr, rows_of
from workloads import CONFIGS, make_contexts, make_lm_weights, make_prefixes, make_set, scaled
from workloads.standin_lm import StandInLM

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _both(w):
    tok, off = make_set(w)
    return tok, off, disc.disc_build_set(tok, off, w.V), oracle.OracleSet(tok, off, w.V)


SET_CASES = [("tiny", {}), ("genret", {}), ("llm", dict(n_draws=200_000)), ("large", dict(n_draws=300_000))]


@pytest.mark.parametrize("name,over", SET_CASES)
def test_sorted_table_and_index_sizes(name, over):
    w = scaled(name, **over)
    tok, off, G, S = _both(w)
    gt, go = disc.disc_set_rows(G)
    st, so = S.rows()
    assert (G.N, G.E, G.l_max) == (S.N, S.E, S.l_max)
    assert np.array_equal(go, so) and np.array_equal(gt, st)
    assert G.n_nodes == S.n_nodes and sum(G.level_nodes) == G.n_nodes
    G.close()


@pytest.mark.parametrize("rows,V,code", [
    ([(1, 2), ()], 4, -2), ([(1, 2), (1, 4)], 4, -3), ([(1, 2), (-1, 0)], 4, -3),
    ([(1, 2), (1, 2, 3)], 4, -4), ([(1, 2, 3), (0,), (1, 2)], 4, -4), ([], 4, -2),
    ([tuple(range(65))], 100, -7),
])
def test_build_rejects_like_the_oracle(rows, V, code):
    with pytest.raises(disc.DiscError) as e:
        disc.disc_build_set(*csr(rows), V)
    assert e.value.code == code
    if code != -7:
        with pytest.raises(oracle.OracleError) as e2:
            oracle.OracleSet(*csr(rows), V)
        assert e2.value.code == code


def test_duplicates_collapse():
    rows = [(3, 1), (0, 2), (3, 1), (0, 1), (3, 0), (0, 2)]
    G = disc.disc_build_set(*csr(rows), 4)
    assert rows_of(*disc.disc_set_rows(G)) == [(0, 1), (0, 2), (3, 0), (3, 1)]


def test_sampling_uniforms_bit_exact():
    seed = 0xDEADBEEF12345678
    for step, row, g0, n in [(0, 0, 0, 1300), (5, 4095, 15_900, 256), (15, 123456, 7, 33)]:
        g = disc.disc_sampling_uniforms(seed, step, row, g0, n).cpu().numpy()
        o = np.array([oracle.group_uniform(seed, step, row, g0 + i) for i in range(n)])
        assert np.array_equal(g.astype(np.float64), o)


def test_mask_with_few_prefixes():
    """Calls with fewer prefixes than the writer has teams of warps, and repeated calls (the row
    counter must come back to zero every time)."""
    w = scaled("llm", n_draws=50_000)
    tok, off, G, S = _both(w)
    prefix, plen = make_prefixes(w, tok, off, 64)
    for n in (1, 2, 5, 6, 7, 13, 25, 64):
        for _ in range(2):
            g = disc.disc_mask(G, torch.as_tensor(prefix[:n], device=DEV), torch.as_tensor(plen[:n], device=DEV))
            m, lo, hi, st = S.mask(prefix[:n], plen[:n])
            assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), m), n
            assert np.array_equal(g["lo"].cpu().numpy(), lo) and np.array_equal(g["hi"].cpu().numpy(), hi)
            assert np.array_equal(g["status"].cpu().numpy(), st)
    G.close()


@pytest.mark.parametrize("name,over,n", [("tiny", {}, 400), ("genret", {}, 3000),
                                          ("llm", dict(n_draws=200_000), 3000),
                                          ("large", dict(n_draws=300_000), 3000),
                                          # rows longer than the writer's shared-memory buffers (W = 4,100 words)
                                          ("large", dict(n_draws=300_000, V=131_200), 2000),
                                          # rows of 128 bytes, the shortest the two-kernel path takes
                                          ("llm", dict(n_draws=50_000, V=1024), 2000),
                                          # a row length that is not a multiple of 16 bytes: the one-kernel path
                                          ("llm", dict(n_draws=100_000, V=32_003), 2000)])
def test_mask_parity(name, over, n):
    w = scaled(name, **over)
    tok, off, G, S = _both(w)
    prefix, plen = make_prefixes(w, tok, off, n)
    rng = np.random.default_rng(5)
    # add complete members, corrupted prefixes and out-of-vocabulary tokens
    extra = n // 10
    r = rng.integers(0, off.shape[0] - 1, extra)
    for j, rr in enumerate(r):
        L = int(off[rr + 1] - off[rr])
        prefix[j, :L] = tok[off[rr]:off[rr + 1]]
        plen[j] = L
    bad = rng.integers(extra, n, extra)
    for j in bad:
        if plen[j] > 0:
            prefix[j, rng.integers(0, plen[j])] = rng.integers(0, w.V)
    prefix[n - 1, 0] = w.V
    plen[n - 1] = max(1, plen[n - 1])
    prefix[n - 2, 0] = -3
    plen[n - 2] = max(1, plen[n - 2])
    g = disc.disc_mask(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV))
    m, lo, hi, st = S.mask(prefix, plen)
    assert np.array_equal(g["status"].cpu().numpy(), st)
    assert np.array_equal(g["lo"].cpu().numpy(), lo) and np.array_equal(g["hi"].cpu().numpy(), hi)
    assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), m)
    assert (st == 1).sum() > 0 and (st == 0).sum() > n // 2
    # the returned cursor continues correctly: a step from it behaves like a step from the prefix
    g2 = disc.disc_mask(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV), want_mask=False)
    assert np.array_equal(g2["node"].cpu().numpy(), g["node"].cpu().numpy())
    G.close()


STEP_CASES = [
    ("tiny", {}, 1.0),
    ("genret", dict(B=64), 1.0),
    ("llm", dict(n_draws=200_000, B=8, K=16, d=64), 1.0),
    ("llm", dict(n_draws=50_000, B=4, K=8, d=64, V=32_003), 0.8),
    ("large", dict(n_draws=300_000, B=8, K=16, d=64), 1.0),
]


@pytest.mark.parametrize("name,over,inv_t", STEP_CASES)
def test_step_lockstep_and_resample(name, over, inv_t):
    w = scaled(name, **over)
    tok, off, G, S = _both(w)
    lm = StandInLM(*make_lm_weights(w), w.logits, DEV)
    ctx = torch.as_tensor(make_contexts(w), device=DEV)
    ls = LockStep(G, S, w.R, with_mask=(w.V <= 40_000))
    prev = ctx.to(torch.int64).repeat_interleave(w.K)
    seed = 20250409 + w.index
    for t in range(G.l_max):
        logits = lm.logits(prev)
        ls.step(logits, t, seed, inv_t)
        prev = torch.where(ls.out.token >= 0, ls.out.token.to(torch.int64), prev)
    assert bool(ls.state.done.all())
    assert ls.near_ties <= max(2, ls.checked // 1000)
    # every decoded sequence is a member
    seqs = {tuple(t for t in s if t >= 0) for s in ls.seq.cpu().numpy().tolist()}
    members = set(rows_of(*S.rows()))
    assert seqs <= members
    # K-way draw on the GPU's log-weights
    logw = ls.state.logw.view(w.B, w.K)
    r = disc.disc_resample(logw, seed=seed, seq_tokens=ls.seq.view(w.B, w.K, -1))
    o = oracle.resample(logw.cpu().numpy(), seed=seed)
    idx = r["idx"].cpu().numpy()
    diff = idx != o["idx"]
    assert np.all(o["gap"][diff] < TOL) and np.all(np.abs(idx[diff] - o["idx"][diff]) == 1)
    assert close(r["logz"].cpu().numpy(), o["logz"]).all()
    assert np.array_equal(r["status"].cpu().numpy(), o["status"])
    picked = ls.seq.view(w.B, w.K, -1).cpu().numpy()[np.arange(w.B), idx]
    assert np.array_equal(r["tokens"].cpu().numpy(), picked)
    print(f"[{name}] rows*steps checked={ls.checked} near-ties={ls.near_ties} max rel logw err={ls.max_err:.2e}")
    G.close()


def _one_step(G, S, logits, prefix_rows, depth, *, seed=3, step=1, inv_t=1.0, with_mask=True):
    """Single step from given prefixes (cursor from disc_mask), compared with the oracle."""
    n = len(depth)
    pre = torch.as_tensor(prefix_rows, device=DEV)
    dep = torch.as_tensor(depth, device=DEV)
    cur = disc.disc_mask(G, pre, dep, want_mask=False)
    st = disc.DiscState(cur["node"].clone(), cur["lo"].clone(), cur["hi"].clone(), dep.clone(),
                        torch.zeros(n, dtype=torch.float32, device=DEV), torch.zeros(n, dtype=torch.uint8, device=DEV))
    out = disc.StepOutputs.empty(n, DEV, mask_words=G.W if with_mask else 0)
    disc.disc_step(G, logits, st, inv_temperature=inv_t, seed=seed, step=step, out=out)
    torch.cuda.synchronize()
    hl, dt = logits_to_host(logits)
    if hl.strides[0] != hl.shape[1] * hl.itemsize:
        hl = np.ascontiguousarray(hl)
    o = S.step(hl, dt, prefix_rows, depth, inv_temperature=inv_t, seed=seed, step=step,
               alt_token=out.token.cpu().numpy())
    return st, out, o


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1001, 4096, 70_001])
def test_step_layouts_and_degenerate_rows(dtype, V):
    """Ragged vocabulary sizes, unaligned rows (scalar path), huge spreads (careful path), -inf / NaN /
    +inf logits, zero allowed mass, rows that are dead or already complete."""
    rng = np.random.default_rng(V)
    L = 4
    n_members = 3000
    rows = np.unique(np.concatenate([rng.integers(0, V, (n_members, L)),
                                     np.stack([np.zeros(V // 2, int), np.arange(0, V - 1, 2)[:V // 2],
                                               np.ones(V // 2, int), np.ones(V // 2, int)], 1)]), axis=0)
    tok, off = csr([tuple(r) for r in rows.tolist()])
    G = disc.disc_build_set(tok, off, V)
    S = oracle.OracleSet(tok, off, V)
    table = rows_of(*S.rows())
    n = 24
    depth = np.array([i % L for i in range(n)], np.int32)
    prefix = np.zeros((n, L), np.int32)
    for i in range(n):
        r = table[int(rng.integers(0, len(table)))]
        prefix[i, :depth[i]] = r[:depth[i]]
    prefix[0, :1] = 0            # the node with V//2 children (dense path) at depth 1
    depth[0] = 1
    prefix[1, :1] = 0
    depth[1] = 1
    # row strides: 16-byte aligned with a ragged tail, exactly V, and an odd stride (scalar path);
    # with and without the mask output (the latter lets small valid sets take the gather path)
    for pad, with_mask in [((-V) % 8, True), ((-V) % 8, False), (0, False), (3, True)]:
        ld = V + pad
        base = (rng.standard_normal((n, ld)) * 2).astype(np.float32)
        base[2] *= 60            # spread far beyond what one fp32 reference covers
        base[3, :] = -1e4
        base[4, rng.integers(0, V, 50)] = -np.inf
        x = torch.as_tensor(base).to(dtype).to(DEV)
        st, out, o = _one_step(G, S, x, prefix, depth, with_mask=with_mask)
        if with_mask:
            m, lo, hi, s0 = S.mask(prefix, depth)
            assert np.array_equal(out.mask.cpu().numpy().view(np.uint32), m)
        assert np.array_equal(out.status.cpu().numpy(), o["status"])
        same = out.token.cpu().numpy() == o["token"]
        assert assert_near_ties(out.token.cpu().numpy()[~same], o, ~same) <= 1
        assert close(st.logw.cpu().numpy(), o["log_mass"]).all(), (st.logw.cpu().numpy(), o["log_mass"])
        assert close(out.logq.cpu().numpy()[same], o["logq"][same]).all()
        assert close(out.logp.cpu().numpy()[same], o["logp"][same]).all()
        assert np.array_equal(st.lo.cpu().numpy()[same], o["lo"][same])
        assert np.array_equal(st.hi.cpu().numpy()[same], o["hi"][same])
        assert np.array_equal(st.done.cpu().numpy()[same], o["done"][same])
    # special values: zero allowed mass, NaN, +inf
    ld = V
    base = (rng.standard_normal((n, ld)) * 2).astype(np.float32)
    allowed0 = np.array(sorted({t[1] for t in table if t[0] == 0}))
    base[0, allowed0] = -np.inf                     # all allowed tokens impossible
    base[1, allowed0[:5]] = -np.inf                 # some allowed tokens impossible
    base[5, 7] = np.nan
    base[6, 9] = np.inf
    x = torch.as_tensor(base).to(dtype).to(DEV)
    st, out, o = _one_step(G, S, x, prefix, depth)
    assert np.array_equal(out.status.cpu().numpy(), o["status"])
    assert out.status[0].item() & disc.ROW_NOMASS and out.token[0].item() == allowed0[0]
    assert out.status[5].item() & disc.ROW_NONFINITE and out.status[6].item() & disc.ROW_NONFINITE
    assert close(st.logw.cpu().numpy(), o["log_mass"]).all()
    same = out.token.cpu().numpy() == o["token"]
    assert same[[0, 1]].all()
    # dead cursor and finished rows leave everything untouched
    st2 = disc.disc_state_init(G, 3, device=DEV)
    st2.node[0] = -1
    st2.done[1] = 1
    keep = st2.clone()
    out2 = disc.disc_step(G, x[:3].contiguous(), st2, seed=1, step=0)
    torch.cuda.synchronize()
    assert out2.token.cpu().tolist()[:2] == [-1, -1]
    assert out2.status.cpu().tolist()[:2] == [disc.ROW_DEAD, disc.ROW_DONE]
    assert torch.equal(st2.logw[:2], keep.logw[:2]) and torch.equal(st2.node[:2], keep.node[:2])
    assert out2.token[2].item() >= 0
    # empty batch
    e = disc.disc_state_init(G, 0, device=DEV)
    disc.disc_step(G, x[:0], e, seed=1, step=0)
    G.close()


def test_argument_errors():
    w = CONFIGS["tiny"]
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    st = disc.disc_state_init(G, 4, device=DEV)
    x = torch.zeros((4, w.V), device=DEV)
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(disc.DiscError) as e:
            disc.disc_step(G, x, st, inv_temperature=bad)
        assert e.value.code == -1
    with pytest.raises(disc.DiscError):
        disc.disc_step(G, x.to(torch.float16), st)
    with pytest.raises(TypeError):
        disc.disc_step(G, x.cpu(), st)
    with pytest.raises(disc.DiscError):
        disc.disc_build_set(tok, off, 0)


@pytest.mark.parametrize("K", [1, 2, 7, 32, 33, 100, 1000])
def test_resample_and_accept_parity(K):
    rng = np.random.default_rng(K)
    B = 3000
    lw = (rng.standard_normal((B, K)) * 3 - 6).astype(np.float32)
    lw[0, :] = -np.inf
    lw[1, :] = -np.inf
    lw[1, K // 2] = -2.0
    lw[2, 0] = np.nan
    lw[3, :] = -50.0
    seq = rng.integers(0, 1000, (B, K, 5)).astype(np.int32)
    t = torch.as_tensor(lw, device=DEV)
    r = disc.disc_resample(t, seed=99, query_base=1000, seq_tokens=torch.as_tensor(seq, device=DEV))
    o = oracle.resample(lw, seed=99, query_ids=np.arange(B) + 1000)
    idx = r["idx"].cpu().numpy()
    diff = idx != o["idx"]
    assert np.all(o["gap"][diff] < TOL) and np.all(np.abs(idx[diff] - o["idx"][diff]) == 1)
    assert diff.sum() <= 3
    assert close(r["logz"].cpu().numpy(), o["logz"]).all()
    assert np.array_equal(r["status"].cpu().numpy(), o["status"])
    assert np.array_equal(r["tokens"].cpu().numpy(), seq[np.arange(B), idx])
    first = disc.disc_accept(t, seed=99, query_base=1000).cpu().numpy()
    fo = oracle.accept(lw, seed=99, query_ids=np.arange(B) + 1000)
    bad = first != fo
    for b in np.nonzero(bad)[0]:      # only a log-weight within fp32 rounding of log(eps) may flip
        k = min(x for x in (first[b], fo[b]) if x >= 0)
        assert abs(float(lw[b, k]) - np.log(oracle.accept_uniform(99, b + 1000, k))) < 1e-5
    assert bad.sum() <= 2


@pytest.mark.parametrize("K", [1, 2, 7, 32, 33, 100])
def test_accept_then_resample_parity(K):
    """disc_accept_resample (Algorithm 1, lines 11-22 on 2K candidates) against the oracle."""
    rng = np.random.default_rng(100 + K)
    B = 3000
    lw = (rng.standard_normal((B, 2 * K)) * 2 - 2).astype(np.float32)
    lw[0, :] = -np.inf                 # nothing acceptable, nothing to weigh
    lw[1, :K] = 0.0                    # the first candidate is always accepted
    lw[2, :K] = -np.inf
    lw[2, K:] = -np.inf
    lw[2, K + K // 2] = -3.0           # a single fresh candidate carries weight
    lw[3, K:] = np.nan
    seq = rng.integers(0, 1000, (B, 2 * K, 4)).astype(np.int32)
    g = disc.disc_accept_resample(torch.as_tensor(lw, device=DEV), seed=7, query_base=50,
                                  seq_tokens=torch.as_tensor(seq, device=DEV))
    o = oracle.accept_resample(lw, seed=7, query_ids=np.arange(B) + 50)
    first, choice = g["first"].cpu().numpy(), g["choice"].cpu().numpy()
    # accept test: only a log-weight within fp32 rounding of log(eps) may flip
    flips = np.nonzero(first != o["first"])[0]
    for b in flips:
        k = min(x for x in (first[b], o["first"][b]) if x >= 0)
        assert abs(float(lw[b, k]) - np.log(oracle.accept_uniform(7, b + 50, k))) < 1e-5
    assert len(flips) <= 2
    same = first == o["first"]
    acc = same & (first >= 0)
    assert np.array_equal(choice[acc], first[acc])
    rej = same & (first < 0)
    diff = rej & (choice != o["choice"])
    assert np.all(o["gap"][diff] < TOL) and np.all(np.abs(choice[diff] - o["choice"][diff]) == 1)
    assert diff.sum() <= 3
    assert np.all((choice[rej] >= K) & (choice[rej] < 2 * K))
    assert (rej.sum() > 0) and (acc.sum() > 0)
    assert close(g["logz"].cpu().numpy(), o["logz"]).all()
    assert np.array_equal(g["status"].cpu().numpy(), o["status"])
    assert np.array_equal(g["tokens"].cpu().numpy(), seq[np.arange(B), choice])


@pytest.mark.parametrize("name,over,n,M", [("tiny", {}, 300, 9), ("genret", {}, 1500, 50),
                                           ("llm", dict(n_draws=200_000), 1500, 50),
                                           ("large", dict(n_draws=300_000), 1200, 100),
                                           ("large", dict(n_draws=300_000), 600, 300),      # one block per prefix, pivots
                                           ("llm", dict(n_draws=200_000), 300, 1000),
                                           ("tiny", {}, 200, 128)])
def test_verify_parity(name, over, n, M):
    """disc_verify (Algorithm 2, lines 4-6: binary search in the sorted array) against the oracle:
    validity, the row every search lands on, the extended mask, the prefix's member range."""
    w = scaled(name, **over)
    tok, off, G, S = _both(w)
    prefix, plen = make_prefixes(w, tok, off, n)
    rng = np.random.default_rng(17)
    # complete members, broken prefixes, tokens outside the vocabulary inside a prefix
    extra = n // 10
    for j, rr in enumerate(rng.integers(0, off.shape[0] - 1, extra)):
        L = int(off[rr + 1] - off[rr])
        prefix[j, :L] = tok[off[rr]:off[rr + 1]]
        plen[j] = L
    for j in rng.integers(extra, n, extra):
        if plen[j] > 0:
            prefix[j, rng.integers(0, plen[j])] = rng.integers(0, w.V)
    prefix[n - 1, 0] = w.V + 5
    plen[n - 1] = max(1, plen[n - 1])
    # candidates: random ids, ids outside [0, V), and for half of the slots a true child
    cand = rng.integers(-2, w.V + 2, (n, M)).astype(np.int32)
    m_true, lo_t, hi_t, st_t = S.mask(prefix, plen)
    for i in range(n):
        bits = np.nonzero(np.unpackbits(m_true[i].view(np.uint8), bitorder="little"))[0]
        if len(bits):
            k = min(M // 2, len(bits))
            cand[i, :k] = rng.choice(bits, k, replace=False)
    g = disc.disc_verify(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV),
                         torch.as_tensor(cand, device=DEV), want_mask=True)
    valid, rows, mask = S.verify(prefix, plen, cand)
    assert np.array_equal(g["valid"].cpu().numpy(), valid)
    assert np.array_equal(g["rows"].cpu().numpy(), rows)
    assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), mask)
    live = st_t == 0
    assert np.array_equal(g["lo"].cpu().numpy()[live], lo_t[live]) and np.array_equal(g["hi"].cpu().numpy()[live], hi_t[live])
    dead = ~live
    assert np.all(g["lo"].cpu().numpy()[dead] == g["hi"].cpu().numpy()[dead])
    assert valid.sum() > n and (valid == 0).sum() > n


def test_verify_with_every_token_a_candidate_gives_disc_masks_mask():
    """M = |V|: the verified mask equals the enumerated one (two independent device paths: the
    sorted table alone against the prefix index)."""
    w = scaled("genret")
    tok, off, G, S = _both(w)
    n = 700
    prefix, plen = make_prefixes(w, tok, off, n)
    pre, ln = torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV)
    cand = torch.arange(w.V, dtype=torch.int32, device=DEV).repeat(n, 1)
    v = disc.disc_verify(G, pre, ln, cand, want_rows=False, want_mask=True)
    m = disc.disc_mask(G, pre, ln)
    assert torch.equal(v["mask"], m["mask"]) and torch.equal(v["lo"], m["lo"]) and torch.equal(v["hi"], m["hi"])
    r = disc.disc_verify(G, pre, ln, cand[:, :0])           # M = 0: ranges only
    assert torch.equal(r["lo"], m["lo"]) and torch.equal(r["hi"], m["hi"])


def test_edge_shapes_threshold_fanouts_maximum_depth_single_member():
    """Fan-outs on both sides of the gather/dense switch (1024 and 1025 children), members of the
    maximum supported length (64 tokens), a set with one member, a batch of one row."""
    V = 2048 + 7
    rows = [(0, b, 5) for b in range(1024)] + [(1, b, 5) for b in range(1025)]
    deep = tuple([2] + [int(x) for x in np.random.default_rng(0).integers(0, V, 62)] + [9])
    rows += [deep, deep[:-1] + (10,)]
    tok, off = csr(rows)
    G = disc.disc_build_set(tok, off, V)
    S = oracle.OracleSet(tok, off, V)
    assert G.l_max == 64 and G.n_heavy == 1
    rng = np.random.default_rng(4)
    for dtype in (torch.float32, torch.bfloat16):
        R = 64
        ls = LockStep(G, S, R, with_mask=True)
        for t in range(G.l_max):
            logits = torch.as_tensor((rng.standard_normal((R, V + 1)) * 3).astype(np.float32)).to(dtype).to(DEV)
            ls.step(logits, t, seed=77)
        assert bool(ls.state.done.all()) and ls.near_ties <= 2
        seqs = {tuple(t for t in s if t >= 0) for s in ls.seq.cpu().numpy().tolist()}
        assert seqs <= set(rows) and any(len(s) == 64 for s in seqs) and any(s[0] == 0 for s in seqs) \
            and any(s[0] == 1 for s in seqs)
    # masks of the two threshold nodes and of the deepest prefixes
    prefix = np.zeros((4, 64), np.int32)
    plen = np.array([1, 1, 63, 64], np.int32)
    prefix[1, 0] = 1
    prefix[2, :63] = deep[:63]
    prefix[3, :64] = deep
    g = disc.disc_mask(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV))
    m, lo, hi, st = S.mask(prefix, plen)
    assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), m)
    assert np.array_equal(g["lo"].cpu().numpy(), lo) and np.array_equal(g["hi"].cpu().numpy(), hi)
    v = disc.disc_verify(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV),
                         torch.as_tensor(np.tile(np.array([0, 5, 9, 10, 1023, 1024, 1025], np.int32), (4, 1)), device=DEV))
    vo, ro, _ = S.verify(prefix, plen, np.tile(np.array([0, 5, 9, 10, 1023, 1024, 1025], np.int32), (4, 1)), want_mask=False)
    assert np.array_equal(v["valid"].cpu().numpy(), vo) and np.array_equal(v["rows"].cpu().numpy(), ro)
    G.close()

    # one member, one row: every step is forced, the weight is that token's probability
    one = [(3, 1, 4, 1, 5)]
    G1 = disc.disc_build_set(*csr(one), 8)
    S1 = oracle.OracleSet(*csr(one), 8)
    ls = LockStep(G1, S1, 1, with_mask=True)
    for t in range(5):
        ls.step(torch.as_tensor(rng.standard_normal((1, 8)).astype(np.float32), device=DEV), t, seed=1)
    assert ls.seq.cpu().numpy().tolist() == [list(one[0])] and bool(ls.state.done.all())
    r = disc.disc_resample(ls.state.logw.view(1, 1), seed=1)
    assert r["idx"].item() == 0 and abs(r["logz"].item() - ls.state.logw.item()) < 1e-6
    G1.close()


def test_nested_members_through_the_end_of_keyword_token():
    """disc_build_set_eok: members that are prefixes of other members (Section 2.1's EOK rule)."""
    rng = np.random.default_rng(21)
    V, EOK = 300, 299
    base = {tuple(int(x) for x in rng.integers(0, V - 1, int(rng.integers(1, 6)))) for _ in range(4000)}
    members = sorted(base | {m[:k] for m in list(base)[:800] for k in range(1, len(m))})
    tok, off = csr(members)
    with pytest.raises(disc.DiscError):
        disc.disc_build_set(tok, off, V)
    G = disc.disc_build_set_eok(tok, off, V, EOK)
    S = oracle.OracleSet(tok, off, V, eok=EOK)
    gt, go = disc.disc_set_rows(G)
    ot, oo = S.rows()
    assert np.array_equal(gt, ot) and np.array_equal(go, oo) and G.N == len(members)
    # masks of prefixes that are members, proper prefixes, and complete (member + EOK)
    n = 600
    prefix = np.zeros((n, G.l_max), np.int32)
    plen = np.zeros(n, np.int32)
    for i in range(n):
        m = members[int(rng.integers(0, len(members)))]
        k = int(rng.integers(0, len(m) + 2))
        seq = (m + (EOK,))[:k]
        prefix[i, :len(seq)] = seq
        plen[i] = len(seq)
    g = disc.disc_mask(G, torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV))
    m, lo, hi, st = S.mask(prefix, plen)
    assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), m) and np.array_equal(g["status"].cpu().numpy(), st)
    assert np.array_equal(g["lo"].cpu().numpy(), lo) and np.array_equal(g["hi"].cpu().numpy(), hi)
    # a lock-step decode: every result is a member followed by EOK
    R = 256
    ls = LockStep(G, S, R, with_mask=True)
    for t in range(G.l_max):
        ls.step(torch.as_tensor((rng.standard_normal((R, V)) * 2).astype(np.float32), device=DEV), t, seed=5)
    assert bool(ls.state.done.all())
    mset = set(members)
    for s in ls.seq.cpu().numpy().tolist():
        s = [t for t in s if t >= 0]
        assert s[-1] == EOK and tuple(s[:-1]) in mset
    with pytest.raises(disc.DiscError):
        disc.disc_build_set_eok(*csr([(1, EOK, 2)]), V, EOK)
    G.close()


def test_step_reads_pinned_host_logits_in_place():
    """The same step with the logits left in pinned host memory gives bit-identical results."""
    w = scaled("llm", n_draws=50_000, B=4, K=8, d=64)
    tok, off, G, S = _both(w)
    rng = np.random.default_rng(2)
    R = w.R
    for dtype in (torch.bfloat16, torch.float32):
        st_a = disc.disc_state_init(G, R, device=DEV)
        st_b = disc.disc_state_init(G, R, device=DEV)
        for t in range(3):
            host = torch.as_tensor((rng.standard_normal((R, w.V)) * 2).astype(np.float32)).to(dtype).pin_memory()
            oa = disc.disc_step(G, host.to(DEV), st_a, seed=9, step=t)
            ob = disc.disc_step(G, host, st_b, seed=9, step=t)
            torch.cuda.synchronize()
            assert torch.equal(oa.token, ob.token) and torch.equal(oa.logq, ob.logq)
            assert torch.equal(st_a.logw, st_b.logw) and torch.equal(st_a.node, st_b.node)
    with pytest.raises(TypeError):
        disc.disc_step(G, torch.zeros((R, w.V), dtype=torch.float32), st_a, seed=9, step=5)   # pageable host memory
    G.close()


def test_sharded_calls_with_row_base_equal_one_call():
    """Query sharding (what N GPUs do): decoding the rows in two calls with row_base / query_base
    set gives bit-identical tokens, log-weights and resampled indices to one call over all rows."""
    w = scaled("llm", n_draws=100_000, B=12, K=8, d=64)
    tok, off, G, S = _both(w)
    lm = StandInLM(*make_lm_weights(w), w.logits, DEV)
    ctx = torch.as_tensor(make_contexts(w), device=DEV)
    R, half = w.R, (w.B // 2) * w.K
    whole = disc.disc_state_init(G, R, device=DEV)
    pa = disc.disc_state_init(G, half, device=DEV)
    pb = disc.disc_state_init(G, R - half, device=DEV)
    seq = torch.full((R, G.l_max), -1, dtype=torch.int32, device=DEV)
    seq_a, seq_b = seq[:half].clone(), seq[half:].clone()
    prev = ctx.to(torch.int64).repeat_interleave(w.K)
    for t in range(G.l_max):
        logits = lm.logits(prev)
        o = disc.disc_step(G, logits, whole, seed=5, step=t, seq_tokens=seq)
        oa = disc.disc_step(G, logits[:half], pa, seed=5, step=t, row_base=0, seq_tokens=seq_a)
        ob = disc.disc_step(G, logits[half:], pb, seed=5, step=t, row_base=half, seq_tokens=seq_b)
        assert torch.equal(o.token, torch.cat([oa.token, ob.token]))
        prev = torch.where(o.token >= 0, o.token.to(torch.int64), prev)
    assert torch.equal(whole.logw, torch.cat([pa.logw, pb.logw])) and torch.equal(seq, torch.cat([seq_a, seq_b]))
    r = disc.disc_resample(whole.logw.view(w.B, w.K), seed=5)
    ra = disc.disc_resample(pa.logw.view(-1, w.K), seed=5, query_base=0)
    rb = disc.disc_resample(pb.logw.view(-1, w.K), seed=5, query_base=w.B // 2)
    assert torch.equal(r["idx"], torch.cat([ra["idx"], rb["idx"]]))
    assert torch.equal(r["logz"], torch.cat([ra["logz"], rb["logz"]]))
    G.close()
