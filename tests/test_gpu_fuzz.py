"""Many small random shapes through the CUDA path against the oracle: vocabularies from 2 tokens,
members of length 1, single-member sets, EOS-closed and fixed-length sets, batches of 1 to 40
rows, fp32 and bf16 logits with aligned and unaligned row strides."""
import numpy as np
import pytest
import torch

import oracle
import paper_2504_09135_b200 as disc
from gpu_helpers import LockStep
from helpers import csr

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _random_set(rng):
    V = int(rng.integers(2, 70))
    L = int(rng.integers(1, 7))
    n = int(rng.integers(1, 200))
    rows = set()
    if rng.random() < 0.5 and V >= 3:
        for _ in range(n):
            ell = int(rng.integers(0, L))
            rows.add(tuple(int(x) for x in rng.integers(0, V - 1, ell)) + (V - 1,))
    else:
        for _ in range(n):
            rows.add(tuple(int(x) for x in rng.integers(0, V, L)))
    return V, sorted(rows)


@pytest.mark.parametrize("block", range(6))
def test_small_random_shapes(block):
    rng = np.random.default_rng(1000 + block)
    for case in range(25):
        V, members = _random_set(rng)
        tok, off = csr(members)
        G = disc.disc_build_set(tok, off, V)
        S = oracle.OracleSet(tok, off, V)
        gt, go = disc.disc_set_rows(G)
        ot, oo = S.rows()
        assert np.array_equal(gt, ot) and np.array_equal(go, oo), (block, case)
        # masks and verification of random prefixes (members' prefixes and arbitrary sequences)
        n = int(rng.integers(1, 40))
        prefix = rng.integers(0, V, (n, G.l_max)).astype(np.int32)
        plen = rng.integers(0, G.l_max + 1, n).astype(np.int32)
        for i in range(n):
            if rng.random() < 0.7:
                m = members[int(rng.integers(0, len(members)))]
                k = int(rng.integers(0, len(m) + 1))
                prefix[i, :k] = m[:k]
                plen[i] = k
        pre, ln = torch.as_tensor(prefix, device=DEV), torch.as_tensor(plen, device=DEV)
        g = disc.disc_mask(G, pre, ln)
        m_o, lo_o, hi_o, st_o = S.mask(prefix, plen)
        assert np.array_equal(g["mask"].cpu().numpy().view(np.uint32), m_o), (block, case)
        assert np.array_equal(g["lo"].cpu().numpy(), lo_o) and np.array_equal(g["hi"].cpu().numpy(), hi_o)
        assert np.array_equal(g["status"].cpu().numpy(), st_o)
        M = int(rng.integers(1, 12))
        cand = rng.integers(-1, V + 1, (n, M)).astype(np.int32)
        v = disc.disc_verify(G, pre, ln, torch.as_tensor(cand, device=DEV), want_mask=True)
        vo, ro, mo = S.verify(prefix, plen, cand)
        assert np.array_equal(v["valid"].cpu().numpy(), vo) and np.array_equal(v["rows"].cpu().numpy(), ro)
        assert np.array_equal(v["mask"].cpu().numpy().view(np.uint32), mo)
        # a lock-step decode
        R = int(rng.integers(1, 40))
        dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
        ld = V + int(rng.integers(0, 9))
        ls = LockStep(G, S, R, with_mask=True)
        for t in range(G.l_max):
            x = torch.as_tensor((rng.standard_normal((R, ld)) * 3).astype(np.float32)).to(dtype).to(DEV)
            ls.step(x, t, seed=block * 100 + case)
        assert bool(ls.state.done.all()), (block, case)
        assert ls.near_ties <= 1
        G.close()
