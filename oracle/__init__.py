"""ctypes loader for the CPU oracle (oracle/disc_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

The shared object is compiled on first use with g++ (a few seconds).
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "disc_oracle.cpp")
_LIB = os.path.join(_HERE, "libdisc_oracle.so")

ERR_ARG, ERR_EMPTY, ERR_TOKEN, ERR_PREFIX, ERR_UNSUPPORTED = -1, -2, -3, -4, -7
F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    with open(_SRC, "rb") as f:
        digest = hashlib.sha256(f.read()).hexdigest()
    try:
        with open(_LIB + ".sha256") as f:
            stale = (not os.path.exists(_LIB)) or f.read().strip() != digest
    except OSError:
        stale = True
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC],
                       check=True)
        os.replace(tmp, _LIB)
        with open(_LIB + ".sha256", "w") as f:
            f.write(digest)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, u32, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64
        L.oracle_build.argtypes = [vp, vp, i64, i32, C.POINTER(vp)]
        L.oracle_build.restype = C.c_int
        L.oracle_free.argtypes = [vp]
        L.oracle_free.restype = None
        L.oracle_info.argtypes = [vp, vp]
        L.oracle_info.restype = None
        L.oracle_rows.argtypes = [vp, vp, vp]
        L.oracle_rows.restype = None
        L.oracle_mask.argtypes = [vp, vp, i32, vp, i64, vp, vp, vp, vp]
        L.oracle_mask.restype = None
        L.oracle_verify.argtypes = [vp, vp, i32, vp, i64, vp, i32, vp, vp, vp]
        L.oracle_verify.restype = None
        L.oracle_step.argtypes = [vp, vp, C.c_int, i64, i64, C.c_float, u64, u32, vp,
                                  vp, i32, vp, vp, vp,
                                  vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_int]
        L.oracle_step.restype = None
        L.oracle_topm.argtypes = [vp, C.c_int, i64, i64, i32, i32, vp]
        L.oracle_topm.restype = None
        L.oracle_step_topm.argtypes = [vp, vp, C.c_int, i64, i64, i32, C.c_float, u64, u32, vp,
                                       vp, i32, vp, vp, vp,
                                       vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_int]
        L.oracle_step_topm.restype = None
        L.oracle_step_plain.argtypes = [vp, vp, C.c_int, i64, i64, C.c_float, u64, u32, vp,
                                        vp, i32, vp, vp,
                                        vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_int]
        L.oracle_step_plain.restype = None
        L.oracle_plain_uniform.argtypes = [u64, u32, u32]
        L.oracle_plain_uniform.restype = C.c_double
        L.oracle_resample.argtypes = [vp, i32, i32, u64, vp, vp, vp, vp, vp, vp]
        L.oracle_resample.restype = None
        L.oracle_accept.argtypes = [vp, i32, i32, u64, vp, vp]
        L.oracle_accept.restype = None
        L.oracle_accept_resample.argtypes = [vp, i32, i32, u64, vp, vp, vp, vp, vp, vp]
        L.oracle_accept_resample.restype = None
        L.oracle_decode_markov.argtypes = [vp, vp, vp, i32, i32, C.c_float, u64, i64,
                                           vp, vp, vp, vp, vp, vp, C.c_int]
        L.oracle_decode_markov.restype = C.c_int
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_philox4x32_10.restype = None
        L.oracle_group_uniform.argtypes = [u64, u32, u32, u32]
        L.oracle_group_uniform.restype = C.c_double
        L.oracle_ingroup_uniform.argtypes = [u64, u32, u32, u32]
        L.oracle_ingroup_uniform.restype = C.c_double
        L.oracle_resample_uniform.argtypes = [u64, u32]
        L.oracle_resample_uniform.restype = C.c_double
        L.oracle_accept_uniform.argtypes = [u64, u32, u32]
        L.oracle_accept_uniform.restype = C.c_double
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle_build failed with code {code}")
        self.code = code


class OracleSet:
    """The constraint set as an explicit prefix tree."""

    def __init__(self, tokens, row_offsets, vocab_size, eok=None):
        """eok: for sets in which a member may be a prefix of another (Section 2.1), the
        end-of-keyword token: every member is closed by it, so that the valid set of a prefix that
        is itself a member contains eok next to the tokens that extend it."""
        tokens = _c(tokens, np.int32)
        row_offsets = _c(row_offsets, np.int64)
        if eok is not None:
            if not 0 <= int(eok) < int(vocab_size) or np.any(tokens == int(eok)):
                raise OracleError(ERR_TOKEN)
            rows = [np.append(tokens[row_offsets[i]:row_offsets[i + 1]], np.int32(eok))
                    for i in range(row_offsets.shape[0] - 1)]
            if any(r.shape[0] == 1 for r in rows):
                raise OracleError(ERR_EMPTY)
            tokens = _c(np.concatenate(rows), np.int32) if rows else tokens
            row_offsets = np.zeros(len(rows) + 1, np.int64)
            row_offsets[1:] = np.cumsum([r.shape[0] for r in rows])
        h = C.c_void_p()
        rc = lib().oracle_build(_p(tokens), _p(row_offsets), row_offsets.shape[0] - 1,
                                int(vocab_size), C.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self._h = h
        info = np.zeros(4, dtype=np.int64)
        lib().oracle_info(self._h, _p(info))
        self.N, self.E, self.l_max, self.n_nodes = (int(x) for x in info)
        self.V = int(vocab_size)
        self.W = (self.V + 31) // 32

    def close(self):
        if getattr(self, "_h", None):
            lib().oracle_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def rows(self):
        """Sorted, de-duplicated table: (tokens int32[E], row_offsets int64[N+1])."""
        tok = np.empty(self.E, dtype=np.int32)
        off = np.empty(self.N + 1, dtype=np.int64)
        lib().oracle_rows(self._h, _p(tok), _p(off))
        return tok, off

    def mask(self, prefix, prefix_len):
        prefix = _c(prefix, np.int32)
        if prefix.ndim == 1:
            prefix = prefix.reshape(1, -1)
        prefix_len = _c(prefix_len, np.int32).reshape(-1)
        n = prefix_len.shape[0]
        ld = prefix.shape[1] if prefix.shape[1] > 0 else 1
        if prefix.shape[1] == 0:
            prefix = np.zeros((n, 1), dtype=np.int32)
        mask = np.empty((n, self.W), dtype=np.uint32)
        lo = np.empty(n, dtype=np.int32)
        hi = np.empty(n, dtype=np.int32)
        status = np.empty(n, dtype=np.uint8)
        lib().oracle_mask(self._h, _p(prefix), ld, _p(prefix_len), n, _p(mask), _p(lo), _p(hi), _p(status))
        return mask, lo, hi, status

    def verify(self, prefix, prefix_len, cand, want_mask=True):
        """Algorithm 2, lines 4-6: validity of M candidate tokens per prefix by binary search in the
        sorted array.  cand int32[n, M] -> (valid uint8[n, M], row_index int32[n, M], mask or None)."""
        prefix = _c(prefix, np.int32)
        if prefix.ndim == 1:
            prefix = prefix.reshape(1, -1)
        prefix_len = _c(prefix_len, np.int32).reshape(-1)
        n = prefix_len.shape[0]
        if prefix.shape[1] == 0:
            prefix = np.zeros((n, 1), dtype=np.int32)
        cand = _c(cand, np.int32).reshape(n, -1)
        M = cand.shape[1]
        valid = np.empty((n, M), np.uint8)
        row_index = np.empty((n, M), np.int32)
        mask = np.empty((n, self.W), np.uint32) if want_mask else None
        lib().oracle_verify(self._h, _p(prefix), prefix.shape[1], _p(prefix_len), n, _p(cand), M, _p(valid),
                            _p(row_index), _p(mask))
        return valid, row_index, mask

    def step(self, logits, dtype, prefix, depth, done=None, *, inv_temperature=1.0, seed=0, step=0,
             row_ids=None, alt_token=None, n_threads=1):
        """One decoding step.  logits: [n, ld] float32 array, or uint16 array holding bf16 bits."""
        depth = _c(depth, np.int32).reshape(-1)
        n = depth.shape[0]
        logits = np.ascontiguousarray(logits)
        assert logits.ndim == 2 and logits.shape[0] == n and logits.shape[1] >= self.V
        assert logits.dtype == (np.float32 if dtype == F32 else np.uint16)
        prefix = _c(prefix, np.int32)
        if prefix.ndim == 1:
            prefix = prefix.reshape(n, -1)
        if prefix.shape[1] == 0:
            prefix = np.zeros((n, 1), dtype=np.int32)
        done = None if done is None else _c(done, np.uint8)
        row_ids = None if row_ids is None else _c(row_ids, np.int64)
        alt_token = None if alt_token is None else _c(alt_token, np.int32)
        o = {
            "token": np.empty(n, np.int32), "lo": np.empty(n, np.int32), "hi": np.empty(n, np.int32),
            "done": np.empty(n, np.uint8), "log_mass": np.empty(n), "lse_all": np.empty(n),
            "lse_ok": np.empty(n), "logq": np.empty(n), "logp": np.empty(n), "best": np.empty(n),
            "second": np.empty(n), "alt": np.empty(n), "ingroup_gap": np.empty(n),
            "n_children": np.empty(n, np.int32),
            "status": np.empty(n, np.uint8),
        }
        lib().oracle_step(self._h, _p(logits), int(dtype), logits.shape[1], n, float(inv_temperature),
                          int(seed), int(step), _p(row_ids), _p(prefix), prefix.shape[1], _p(depth),
                          _p(done), _p(alt_token),
                          _p(o["token"]), _p(o["lo"]), _p(o["hi"]), _p(o["done"]), _p(o["log_mass"]),
                          _p(o["lse_all"]), _p(o["lse_ok"]), _p(o["logq"]), _p(o["logp"]),
                          _p(o["best"]), _p(o["second"]), _p(o["alt"]), _p(o["ingroup_gap"]), _p(o["n_children"]),
                          _p(o["status"]), int(n_threads))
        return o

    def step_topm(self, logits, dtype, M, prefix, depth, done=None, *, inv_temperature=1.0, seed=0, step=0,
                  row_ids=None, alt_token=None, n_threads=1):
        """One decoding step in the paper's top-M mode: the M most probable tokens are verified against
        the sorted array (Algorithm 2) and the token is drawn among the verified ones.  Outputs as for
        step(), with n_children = the number of verified candidates; a row without any gets status 1."""
        depth = _c(depth, np.int32).reshape(-1)
        n = depth.shape[0]
        logits = np.ascontiguousarray(logits)
        assert logits.ndim == 2 and logits.shape[0] == n and logits.shape[1] >= self.V
        assert logits.dtype == (np.float32 if dtype == F32 else np.uint16)
        prefix = _c(prefix, np.int32)
        if prefix.ndim == 1:
            prefix = prefix.reshape(n, -1)
        if prefix.shape[1] == 0:
            prefix = np.zeros((n, 1), dtype=np.int32)
        done = None if done is None else _c(done, np.uint8)
        row_ids = None if row_ids is None else _c(row_ids, np.int64)
        alt_token = None if alt_token is None else _c(alt_token, np.int32)
        o = {
            "token": np.empty(n, np.int32), "lo": np.empty(n, np.int32), "hi": np.empty(n, np.int32),
            "done": np.empty(n, np.uint8), "log_mass": np.empty(n), "lse_all": np.empty(n),
            "lse_ok": np.empty(n), "logq": np.empty(n), "logp": np.empty(n), "best": np.empty(n),
            "second": np.empty(n), "alt": np.empty(n), "ingroup_gap": np.empty(n),
            "n_children": np.empty(n, np.int32),
            "status": np.empty(n, np.uint8),
        }
        lib().oracle_step_topm(self._h, _p(logits), int(dtype), logits.shape[1], n, int(M), float(inv_temperature),
                               int(seed), int(step), _p(row_ids), _p(prefix), prefix.shape[1], _p(depth),
                               _p(done), _p(alt_token),
                               _p(o["token"]), _p(o["lo"]), _p(o["hi"]), _p(o["done"]), _p(o["log_mass"]),
                               _p(o["lse_all"]), _p(o["lse_ok"]), _p(o["logq"]), _p(o["logp"]),
                               _p(o["best"]), _p(o["second"]), _p(o["alt"]), _p(o["ingroup_gap"]), _p(o["n_children"]),
                               _p(o["status"]), int(n_threads))
        return o

    def step_plain(self, logits, dtype, prefix, depth, done=None, *, inv_temperature=1.0, seed=0, step=0,
                   row_ids=None, n_threads=1):
        """The same step with the plain sampler: inverse CDF over the allowed tokens in ascending id,
        one uniform per (row, step).  Everything but the token (and logq / logp / range / done, which
        follow the token) equals step()'s."""
        depth = _c(depth, np.int32).reshape(-1)
        n = depth.shape[0]
        logits = np.ascontiguousarray(logits)
        assert logits.ndim == 2 and logits.shape[0] == n and logits.shape[1] >= self.V
        assert logits.dtype == (np.float32 if dtype == F32 else np.uint16)
        prefix = _c(prefix, np.int32)
        if prefix.ndim == 1:
            prefix = prefix.reshape(n, -1)
        if prefix.shape[1] == 0:
            prefix = np.zeros((n, 1), dtype=np.int32)
        done = None if done is None else _c(done, np.uint8)
        row_ids = None if row_ids is None else _c(row_ids, np.int64)
        o = {"token": np.empty(n, np.int32), "lo": np.empty(n, np.int32), "hi": np.empty(n, np.int32),
             "done": np.empty(n, np.uint8), "log_mass": np.empty(n), "lse_all": np.empty(n),
             "lse_ok": np.empty(n), "logq": np.empty(n), "logp": np.empty(n), "status": np.empty(n, np.uint8)}
        lib().oracle_step_plain(self._h, _p(logits), int(dtype), logits.shape[1], n, float(inv_temperature),
                                int(seed), int(step), _p(row_ids), _p(prefix), prefix.shape[1], _p(depth), _p(done),
                                _p(o["token"]), _p(o["lo"]), _p(o["hi"]), _p(o["done"]), _p(o["log_mass"]),
                                _p(o["lse_all"]), _p(o["lse_ok"]), _p(o["logq"]), _p(o["logp"]), _p(o["status"]),
                                int(n_threads))
        return o

    def decode_markov(self, Z, ctx, K, *, inv_temperature=1.0, seed=0, query_base=0, n_threads=1):
        """Free-running SampleCandidate x (B*K) + K-way draw under a Markov LM table Z[V, V]."""
        Z = _c(Z, np.float32)
        assert Z.shape == (Z.shape[0], self.V)
        ctx = _c(ctx, np.int32)
        B = ctx.shape[0]
        L = self.l_max
        o = {
            "seq": np.empty((B, K, L), np.int32), "len": np.empty((B, K), np.int32),
            "logw": np.empty((B, K)), "logw32": np.empty((B, K), np.float32),
            "idx": np.empty(B, np.int32), "logz": np.empty(B),
        }
        rc = lib().oracle_decode_markov(self._h, _p(Z), _p(ctx), B, K, float(inv_temperature), int(seed),
                                        int(query_base), _p(o["seq"]), _p(o["len"]), _p(o["logw"]),
                                        _p(o["logw32"]), _p(o["idx"]), _p(o["logz"]), int(n_threads))
        assert rc == 0
        return o


def topm(logits, dtype, V, M):
    """Algorithm 2, line 3: the M largest logits of every row (lower id first among equals, NaN last),
    as token ids in ascending order; int32[n, M], -1 padded when M > V."""
    logits = np.ascontiguousarray(logits)
    n = logits.shape[0]
    cand = np.empty((n, int(M)), np.int32)
    lib().oracle_topm(_p(logits), int(dtype), logits.shape[1], n, int(V), int(M), _p(cand))
    return cand


def resample(logw, seed=0, query_ids=None):
    logw = _c(logw, np.float32)
    B, K = logw.shape
    query_ids = None if query_ids is None else _c(query_ids, np.int64)
    o = {"idx": np.empty(B, np.int32), "logz": np.empty(B), "u": np.empty(B), "gap": np.empty(B),
         "status": np.empty(B, np.uint8)}
    lib().oracle_resample(_p(logw), B, K, int(seed), _p(query_ids), _p(o["idx"]), _p(o["logz"]),
                          _p(o["u"]), _p(o["gap"]), _p(o["status"]))
    return o


def accept(logw, seed=0, query_ids=None):
    logw = _c(logw, np.float32)
    B, K = logw.shape
    query_ids = None if query_ids is None else _c(query_ids, np.int64)
    out = np.empty(B, np.int32)
    lib().oracle_accept(_p(logw), B, K, int(seed), _p(query_ids), _p(out))
    return out


def accept_resample(logw, seed=0, query_ids=None):
    """Algorithm 1, lines 11-22 on [B][2K] log-weights: the first K columns are tried in order by
    the accept test, the last K are the fresh candidates of the K-way draw."""
    logw = _c(logw, np.float32)
    B, K2 = logw.shape
    assert K2 % 2 == 0 and K2 > 0
    query_ids = None if query_ids is None else _c(query_ids, np.int64)
    o = {"choice": np.empty(B, np.int32), "first": np.empty(B, np.int32), "logz": np.empty(B),
         "gap": np.empty(B), "status": np.empty(B, np.uint8)}
    lib().oracle_accept_resample(_p(logw), B, K2 // 2, int(seed), _p(query_ids), _p(o["choice"]), _p(o["first"]),
                                 _p(o["logz"]), _p(o["gap"]), _p(o["status"]))
    return o


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def group_uniform(seed, step, row, group):
    """Uniform behind the Gumbel noise of token group `group` (= token id >> 3)."""
    return lib().oracle_group_uniform(int(seed), int(step), int(row), int(group))


def ingroup_uniform(seed, step, row, group):
    """Uniform of the inverse-CDF draw inside the winning group."""
    return lib().oracle_ingroup_uniform(int(seed), int(step), int(row), int(group))


def plain_uniform(seed, step, row):
    """Uniform of the plain inverse-CDF sampler for (row, step)."""
    return lib().oracle_plain_uniform(int(seed), int(step), int(row))


def resample_uniform(seed, query):
    return lib().oracle_resample_uniform(int(seed), int(query))


def accept_uniform(seed, query, k):
    return lib().oracle_accept_uniform(int(seed), int(query), int(k))
