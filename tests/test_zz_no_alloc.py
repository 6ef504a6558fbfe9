"""disc_mask_static (the entry point that allocates nothing) against disc_mask and against the CPU
oracle, through the C ABI.

Named so that it is collected after the other GPU tests: it must pass both alone and with whatever
the earlier tests left on the device and in the library's static word block."""
import numpy as np
import pytest
import torch

import oracle
from workloads import make_prefixes, make_set, scaled

pytestmark = pytest.mark.gpu


def _prefixes(w, tok, off, n, seed):
    prefix, plen = make_prefixes(w, tok, off, n)
    rng = np.random.default_rng(seed)
    # a different mix on every call: shuffle, then break a few prefixes and complete a few others
    order = rng.permutation(n)
    prefix, plen = prefix[order].copy(), plen[order].copy()
    for j in rng.integers(0, n, n // 16):
        if plen[j] > 0:
            prefix[j, rng.integers(0, plen[j])] = rng.integers(0, w.V)
    for j, r in zip(rng.integers(0, n, n // 16), rng.integers(0, off.shape[0] - 1, n // 16)):
        L = int(off[r + 1] - off[r])
        prefix[j, :L] = tok[off[r]:off[r + 1]]
        plen[j] = L
    return prefix, plen


@pytest.mark.parametrize("name,over,n", [("llm", dict(n_draws=200_000), 3000), ("tiny", {}, 257),
                                         ("large", dict(n_draws=300_000), 1500)])
def test_static_entry_point_matches_disc_mask_on_two_calls_in_a_row(name, over, n):
    import paper_2504_09135_b200 as disc
    dev = torch.device("cuda", 0)
    w = scaled(name, **over)
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        pairs = []
        for call in range(2):
            prefix, plen = _prefixes(w, tok, off, n + 17 * call, seed=11 + call)
            pre, ln = torch.as_tensor(prefix, device=dev), torch.as_tensor(plen, device=dev)
            ref = disc.disc_mask(G, pre, ln)
            out = {k: torch.full_like(v, 7) for k, v in ref.items()}       # outputs pre-filled with junk
            pairs.append((ref, out, pre, ln))
        torch.cuda.synchronize()
        # the two calls under test, back to back on one stream, nothing in between
        for ref, out, pre, ln in pairs:
            disc.disc_mask_static(G, pre, ln, out=out)
        torch.cuda.synchronize()
        S = oracle.OracleSet(tok, off, w.V)
        for ref, out, pre, ln in pairs:
            for key in ("mask", "lo", "hi", "node", "status"):
                assert torch.equal(ref[key], out[key]), key
            # and against the oracle's prefix tree, so that a fault common to both CUDA entry
            # points cannot pass
            m, lo, hi, st = S.mask(pre.cpu().numpy(), ln.cpu().numpy())
            assert np.array_equal(out["mask"].cpu().numpy().view(np.uint32), m)
            assert np.array_equal(out["lo"].cpu().numpy(), lo) and np.array_equal(out["hi"].cpu().numpy(), hi)
            assert np.array_equal(out["status"].cpu().numpy(), st)
        S.close()
        # ranges only (no mask output) go through the same entry point
        ref, _, pre, ln = pairs[0]
        r2 = disc.disc_mask_static(G, pre, ln, want_mask=False)
        assert r2["mask"] is None and torch.equal(r2["lo"], ref["lo"]) and torch.equal(r2["status"], ref["status"])
        # the promise of the entry point: with the outputs preallocated, a call takes no device memory
        ref, out, pre, ln = pairs[1]
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        for _ in range(2):
            disc.disc_mask_static(G, pre, ln, out=out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
    finally:
        G.close()


def test_static_entry_point_rejects_sizes_beyond_its_limit():
    import ctypes as C

    import paper_2504_09135_b200 as disc
    from paper_2504_09135_b200 import binding
    dev = torch.device("cuda", 0)
    w = scaled("tiny")
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    try:
        one = torch.zeros(1, dtype=torch.int32, device=dev)
        st = torch.zeros(1, dtype=torch.uint8, device=dev)
        # the size check comes before any pointer is used, so a one-element buffer is enough
        rc = binding.lib().disc_mask_static(G.handle, 0, 0, one.data_ptr(), C.c_int64(binding.MASK_STATIC_MAX_ROWS + 1),
                                            0, 0, 0, 0, st.data_ptr(), 0)
        assert rc == -7
        assert b"unsupported" in binding.lib().disc_error_string(rc)
        with pytest.raises(ValueError):
            disc.disc_mask_static(G, torch.zeros((0, 1), dtype=torch.int32, device=dev),
                                  torch.empty(binding.MASK_STATIC_MAX_ROWS + 1, dtype=torch.int32, device="meta"))
    finally:
        G.close()
