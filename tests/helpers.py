"""Small brute-force helpers for the tests (no method code from oracle/ or the CUDA path)."""
import numpy as np
from scipy.special import log_softmax


def csr(rows):
    tok = np.array([t for r in rows for t in r], dtype=np.int32)
    off = np.zeros(len(rows) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(r) for r in rows])
    return tok, off


def rows_of(tok, off):
    return [tuple(int(x) for x in tok[off[i]:off[i + 1]]) for i in range(len(off) - 1)]


def is_prefix(a, s):
    return len(a) <= len(s) and tuple(s[:len(a)]) == tuple(a)


def valid_set(members, a, V):
    """A_{a,S} by scanning every member (Section 2.1)."""
    a = tuple(a)
    return sorted({s[len(a)] for s in members if len(s) > len(a) and s[:len(a)] == a})


def bits(mask_row, V):
    return {v for v in range(V) if (int(mask_row[v >> 5]) >> (v & 31)) & 1}


def f32_to_bf16_bits(x):
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    import torch
    t = torch.as_tensor(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def exact_member_tables(members, Z, ctx, V, inv_t=1.0):
    """For a first-order Markov LM with logits table Z (rows: previous token; the first step uses
    the context token), by enumeration in fp64:
        logP[a]  = log P_L(a)                       (product of conditionals)
        logx[a]  = log x(a) = sum_i log P_L(A_{a<i,S} | a<i)        (Appendix A)
    """
    members = [tuple(m) for m in members]
    LS = log_softmax(np.asarray(Z, dtype=np.float64) * inv_t, axis=1)
    logP = np.zeros(len(members))
    logx = np.zeros(len(members))
    cache = {}
    for j, a in enumerate(members):
        prev = ctx
        for i, t in enumerate(a):
            pre = a[:i]
            if (pre, prev) not in cache:
                A = valid_set(members, pre, V)
                cache[(pre, prev)] = np.logaddexp.reduce(LS[prev, A])
            logx[j] += cache[(pre, prev)]
            logP[j] += LS[prev, t]
            prev = t
    return logP, logx


def tv(p, q):
    return 0.5 * float(np.abs(np.asarray(p) - np.asarray(q)).sum())
