"""Seeded generators for the five synthetic workloads.

Shapes follow the paper's task statistics (Table "Task Statistics": corpora of
4.6-5.9 M members, 7.7-9.5 tokens on average, vocabularies of 50,264 and
128,256; Section 4.1: batch size 128, temperature 1).  The paper's corpora and
models are not available, so every input is drawn from a seeded numpy
generator; nothing here reproduces an item of any dataset.

Only inputs are produced here.  No function in this module computes a mask,
a softmax, a sample or a weight.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass

import numpy as np

BASE_SEED = 250409135


@dataclass(frozen=True)
class Workload:
    """One synthetic workload.

    name        label used in logs
    index       position of its seed stream under BASE_SEED
    V           vocabulary size
    n_draws     number of member sequences drawn (before de-duplication)
    len_min/len_max  member length range, inclusive; includes the EOS token
                when `eos` is true
    eos         close every member with token V-1 (needed for variable lengths
                so that no member is a proper prefix of another)
    token_dist  "uniform" or "zipf" (rank r has probability ~ r**-zipf_s, ranks
                mapped to ids by a seeded permutation)
    distinct    redraw until all n_draws members are distinct
    B, K        queries and candidates per query
    d           hidden width of the stand-in language model
    logits      "f32" or "bf16"
    bias        stand-in LM has a bias vector
    w_std       "one" -> W ~ N(0,1);  "inv_sqrt_d" -> W ~ N(0,1/d)
    n_prefixes  number of prefixes for the mask-only workload (0 = none)
    """
    name: str
    index: int
    V: int
    n_draws: int
    len_min: int
    len_max: int
    eos: bool
    token_dist: str
    distinct: bool
    B: int
    K: int
    d: int
    logits: str
    bias: bool
    w_std: str
    zipf_s: float = 1.1
    n_prefixes: int = 0

    @property
    def R(self) -> int:
        return self.B * self.K


CONFIGS = {
    "tiny": Workload("tiny", 0, V=64, n_draws=256, len_min=3, len_max=3, eos=False,
                     token_dist="uniform", distinct=True, B=4, K=4, d=32,
                     logits="f32", bias=True, w_std="one"),
    "genret": Workload("genret", 1, V=256, n_draws=100_000, len_min=4, len_max=4, eos=False,
                       token_dist="uniform", distinct=True, B=256, K=8, d=256,
                       logits="bf16", bias=False, w_std="inv_sqrt_d"),
    "llm": Workload("llm", 2, V=32_000, n_draws=1_000_000, len_min=8, len_max=8, eos=False,
                    token_dist="zipf", distinct=False, B=64, K=16, d=1024,
                    logits="bf16", bias=False, w_std="inv_sqrt_d"),
    "large": Workload("large", 3, V=128_256, n_draws=10_000_000, len_min=4, len_max=16, eos=True,
                      token_dist="zipf", distinct=False, B=128, K=32, d=2048,
                      logits="bf16", bias=False, w_std="inv_sqrt_d"),
    # the mask-only stress shares the "large" constraint table (same seed stream)
    "mask": Workload("mask", 3, V=128_256, n_draws=10_000_000, len_min=4, len_max=16, eos=True,
                     token_dist="zipf", distinct=False, B=128, K=32, d=2048,
                     logits="bf16", bias=False, w_std="inv_sqrt_d", n_prefixes=65_536),
}


def scaled(name: str, **overrides) -> Workload:
    """A config with some fields replaced (smaller sets for tests)."""
    return dataclasses.replace(CONFIGS[name], **overrides)


def _streams(w: Workload, salt: int = 0):
    """Independent generators for (set, contexts, prefixes, lm weights)."""
    root = np.random.SeedSequence(BASE_SEED + salt).spawn(5)[w.index]
    return [np.random.Generator(np.random.PCG64(s)) for s in root.spawn(4)]


def _zipf_ids(rng, n: int, n_ids: int, s: float, perm: np.ndarray) -> np.ndarray:
    """n draws of a rank with P(rank r) ~ (r+1)**-s over n_ids ranks, mapped by perm."""
    p = np.arange(1, n_ids + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p)
    cdf /= cdf[-1]
    out = np.empty(n, dtype=np.int32)
    chunk = 1 << 23
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        u = rng.random(b - a)
        r = np.searchsorted(cdf, u, side="right")
        np.minimum(r, n_ids - 1, out=r)
        out[a:b] = perm[r]
    return out


def make_set(w: Workload, salt: int = 0):
    """Draw the constraint set.  Returns (tokens int32[E], row_offsets int64[n+1]).

    Rows come in draw order: unsorted, and for the zipf workloads possibly with
    duplicates (the builders de-duplicate and report the final size).
    """
    rng = _streams(w, salt)[0]
    n = w.n_draws
    eos_id = w.V - 1
    n_ids = w.V - 1 if w.eos else w.V
    if w.len_min == w.len_max:
        lens = np.full(n, w.len_min, dtype=np.int64)
    else:
        lens = rng.integers(w.len_min, w.len_max + 1, size=n, dtype=np.int64)
    row_off = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(lens, out=row_off[1:])
    E = int(row_off[-1])

    if w.distinct:
        if w.len_min != w.len_max or w.eos:
            raise ValueError("distinct sets are fixed-length without EOS")
        L = w.len_min
        if n > n_ids ** L:
            raise ValueError("more distinct members requested than exist")
        have = np.empty((0, L), dtype=np.int32)
        while have.shape[0] < n:
            draw = rng.integers(0, n_ids, size=(int(n * 1.25) + 16, L), dtype=np.int32)
            have = np.unique(np.concatenate([have, draw]), axis=0)
        rows = have[rng.permutation(have.shape[0])[:n]]
        return np.ascontiguousarray(rows.reshape(-1)), row_off

    if w.token_dist == "uniform":
        tokens = rng.integers(0, n_ids, size=E, dtype=np.int32)
    elif w.token_dist == "zipf":
        perm = rng.permutation(n_ids).astype(np.int32)
        tokens = _zipf_ids(rng, E, n_ids, w.zipf_s, perm)
    else:
        raise ValueError(w.token_dist)
    if w.eos:
        tokens[row_off[1:] - 1] = eos_id
    return tokens, row_off


def make_contexts(w: Workload, salt: int = 0) -> np.ndarray:
    """Per-query context token fed to the stand-in LM at the first step, int32[B]."""
    rng = _streams(w, salt)[1]
    return rng.integers(0, w.V, size=w.B, dtype=np.int32)


def make_prefixes(w: Workload, tokens: np.ndarray, row_off: np.ndarray, n: int | None = None,
                  salt: int = 0):
    """Prefixes of members cut at uniform random depths.

    Row r ~ U[0, rows), depth delta ~ U{0 .. len_r - 1}; the prefix is the first
    delta tokens of row r (never a complete member; delta = 0 is the empty prefix).
    Returns (prefix int32[n, len_max] zero-padded, prefix_len int32[n]).
    """
    rng = _streams(w, salt)[2]
    n = w.n_prefixes if n is None else n
    n_rows = row_off.shape[0] - 1
    r = rng.integers(0, n_rows, size=n)
    lens = (row_off[r + 1] - row_off[r]).astype(np.int64)
    delta = (rng.random(n) * lens).astype(np.int64)
    np.minimum(delta, lens - 1, out=delta)
    ld = int(w.len_max)
    prefix = np.zeros((n, ld), dtype=np.int32)
    pos = np.arange(ld, dtype=np.int64)[None, :]
    take = pos < delta[:, None]
    src = row_off[r][:, None] + pos
    prefix[take] = tokens[src[take]]
    return prefix, delta.astype(np.int32)


def make_lm_weights(w: Workload, salt: int = 0):
    """Stand-in LM parameters: E (V x d), W (d x V), b (V) or None, float32.

    logits(prev) = E[prev] @ W (+ b): a first-order Markov model, so the exact
    sequence probabilities needed by the tests are products of table look-ups.
    """
    rng = _streams(w, salt)[3]
    E = rng.standard_normal((w.V, w.d), dtype=np.float32)
    W = rng.standard_normal((w.d, w.V), dtype=np.float32)
    if w.w_std == "inv_sqrt_d":
        W *= np.float32(1.0 / np.sqrt(w.d))
    b = rng.standard_normal(w.V, dtype=np.float32) if w.bias else None
    return E, W, b
