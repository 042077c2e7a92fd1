"""ctypes front end of the CPU oracle (``sdms_oracle.cpp``).

TEST INFRASTRUCTURE ONLY.  Imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark; the CUDA library and its Python binding
never import it.  ``build()`` compiles the C++ file with g++; nothing else is
needed to use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdms_oracle.cpp")
_LIB = os.path.join(_HERE, "libsdms_oracle.so")
_lib = None

ST_BAD_COUNT, ST_CAPACITY, ST_BAD_TOKEN, ST_BAD_LOGPROB = 1, 2, 4, 8


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
                               "-pthread", _SRC, "-o", _LIB])
    return _LIB


def _ptr(a, typ):
    return a.ctypes.data_as(C.POINTER(typ))


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        l.orc_create.restype = C.c_void_p
        l.orc_create.argtypes = [C.c_int] * 5 + [C.c_float, C.c_int]
        l.orc_destroy.argtypes = [C.c_void_p]
        l.orc_prob_to_fixed.restype = C.c_int32
        l.orc_prob_to_fixed.argtypes = [C.c_float]
        l.orc_weight.restype = C.c_double
        l.orc_weight.argtypes = [C.c_float, C.c_int64, C.c_int64]
        for name in ("orc_append", "orc_append_fixed", "orc_accept_commit", "orc_trim"):
            getattr(l, name).restype = C.c_uint32
        l.orc_num_matches.restype = C.c_int
        l.orc_edit_distance.restype = C.c_int
        l.orc_get_draft.restype = C.c_int
        l.orc_build_beams.restype = C.c_int
        _lib = l
    return _lib


def prob_to_fixed(lp: float) -> int:
    return int(lib().orc_prob_to_fixed(C.c_float(lp)))


def edit_distance(a, b) -> int:
    a = np.ascontiguousarray(a, dtype=np.int32); b = np.ascontiguousarray(b, dtype=np.int32)
    return int(lib().orc_edit_distance(_ptr(a, C.c_int32), C.c_int(len(a)), _ptr(b, C.c_int32), C.c_int(len(b))))


def weight(alpha: float, S: int, cnt: int) -> float:
    return float(lib().orc_weight(C.c_float(alpha), C.c_int64(S), C.c_int64(cnt)))


class Oracle:
    """State of G prompts x N paths and the per-path draft construction."""

    def __init__(self, G, N, L, V, D, alpha=1.0, mode=0, eps=0, pool=0, max_matches=0):
        self.G, self.N, self.L, self.V, self.D = G, N, L, V, D
        self.eps, self.pool, self.max_matches = eps, pool, max_matches
        self.P = G * N
        self.alpha, self.mode = alpha, mode
        self._l = lib()
        self._h = C.c_void_p(self._l.orc_create(G, N, L, V, D, C.c_float(alpha), mode))
        self._l.orc_set_epsilon(self._h, C.c_int(eps))
        self._l.orc_set_pool(self._h, C.c_int(pool))
        self._l.orc_set_max_matches(self._h, C.c_int(max_matches))

    def __del__(self):
        if getattr(self, "_h", None):
            self._l.orc_destroy(self._h)
            self._h = None

    # -- state -----------------------------------------------------------
    def append(self, tokens, logprobs, counts) -> int:
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        logprobs = np.ascontiguousarray(logprobs, dtype=np.float32)
        counts = np.ascontiguousarray(counts, dtype=np.int32)
        assert tokens.shape == logprobs.shape and tokens.shape[0] == self.P
        return int(self._l.orc_append(self._h, _ptr(tokens, C.c_int32), _ptr(logprobs, C.c_float),
                                      _ptr(counts, C.c_int32), C.c_int(tokens.shape[1])))

    def append_fixed(self, tokens, pq, counts) -> int:
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        pq = np.ascontiguousarray(pq, dtype=np.int32)
        counts = np.ascontiguousarray(counts, dtype=np.int32)
        return int(self._l.orc_append_fixed(self._h, _ptr(tokens, C.c_int32), _ptr(pq, C.c_int32),
                                            _ptr(counts, C.c_int32), C.c_int(tokens.shape[1])))

    def trim(self, keep) -> int:
        keep = np.ascontiguousarray(keep, dtype=np.int32)
        assert keep.shape == (self.P,)
        return int(self._l.orc_trim(self._h, _ptr(keep, C.c_int32)))

    def lengths(self) -> np.ndarray:
        out = np.zeros(self.P, dtype=np.int32)
        self._l.orc_get_lengths(self._h, _ptr(out, C.c_int32))
        return out

    def history(self, p):
        n = int(self.lengths()[p])
        tok = np.zeros(max(n, 1), dtype=np.int32)
        pq = np.zeros(max(n, 1), dtype=np.int32)
        self._l.orc_get_history(self._h, C.c_int(p), _ptr(tok, C.c_int32), _ptr(pq, C.c_int32))
        return tok[:n], pq[:n]

    # -- draft construction ------------------------------------------------
    def build_path(self, k, i):
        self._l.orc_build_path(self._h, C.c_int(k), C.c_int(i))

    def build_all(self, k, nthreads=1):
        self._l.orc_build_all(self._h, C.c_int(k), C.c_int(nthreads))

    def matches(self, i) -> np.ndarray:
        n = self._l.orc_num_matches(self._h, C.c_int(i))
        out = np.zeros(max(n, 1), dtype=np.int32)
        self._l.orc_get_matches(self._h, C.c_int(i), _ptr(out, C.c_int32))
        return out[:n]

    def layer(self, i, d):
        """Nodes {tok: (S, cnt)} and edges {(u, v): (S, cnt)} of layer d (1-based)."""
        nn, ne = C.c_int32(0), C.c_int32(0)
        self._l.orc_layer_counts(self._h, C.c_int(i), C.c_int(d), C.byref(nn), C.byref(ne))
        nn, ne = nn.value, ne.value
        tok = np.zeros(max(nn, 1), np.int32); S = np.zeros(max(nn, 1), np.int64); cnt = np.zeros(max(nn, 1), np.int64)
        self._l.orc_get_nodes(self._h, C.c_int(i), C.c_int(d), _ptr(tok, C.c_int32), _ptr(S, C.c_int64), _ptr(cnt, C.c_int64))
        nodes = {int(tok[x]): (int(S[x]), int(cnt[x])) for x in range(nn)}
        u = np.zeros(max(ne, 1), np.int32); v = np.zeros(max(ne, 1), np.int32)
        S = np.zeros(max(ne, 1), np.int64); cnt = np.zeros(max(ne, 1), np.int64)
        self._l.orc_get_edges(self._h, C.c_int(i), C.c_int(d), _ptr(u, C.c_int32), _ptr(v, C.c_int32),
                              _ptr(S, C.c_int64), _ptr(cnt, C.c_int64))
        edges = {(int(u[x]), int(v[x])): (int(S[x]), int(cnt[x])) for x in range(ne)}
        return nodes, edges

    def draft(self, i):
        tok = np.zeros(self.D, np.int32); sc = np.zeros(self.D); ew = np.zeros(self.D)
        n = self._l.orc_get_draft(self._h, C.c_int(i), _ptr(tok, C.c_int32), _ptr(sc, C.c_double), _ptr(ew, C.c_double))
        return tok[:n].copy(), sc[:n].copy(), ew[:n].copy()

    def beams(self, i, B):
        """The B best paths of the pool of path i's last build: (tokens [n][<=D] as lists, values [n])."""
        tok = np.full((B, self.D), -1, np.int32); ln = np.zeros(B, np.int32); val = np.zeros(B)
        n = self._l.orc_build_beams(self._h, C.c_int(i), C.c_int(B), _ptr(tok, C.c_int32), _ptr(ln, C.c_int32),
                                    _ptr(val, C.c_double))
        return [tok[b, :ln[b]].tolist() for b in range(n)], val[:n].copy()

    def drafts(self):
        tok = np.zeros((self.P, self.D), np.int32); ln = np.zeros(self.P, np.int32)
        sc = np.zeros((self.P, self.D), np.float32); ew = np.zeros((self.P, self.D), np.float32)
        self._l.orc_get_drafts(self._h, _ptr(tok, C.c_int32), _ptr(ln, C.c_int32), _ptr(sc, C.c_float), _ptr(ew, C.c_float))
        return tok, ln, sc, ew

    def export(self, i, B, Ke):
        D = self.D
        r = dict(node_tok=np.zeros((D, B), np.int32), node_S=np.zeros((D, B), np.int64),
                 node_cnt=np.zeros((D, B), np.int32), node_count=np.zeros(D, np.int32),
                 edge_dst=np.zeros((D, B, Ke), np.int32), edge_S=np.zeros((D, B, Ke), np.int64),
                 edge_cnt=np.zeros((D, B, Ke), np.int32), out_degree=np.zeros((D, B), np.int32))
        self._l.orc_get_export(self._h, C.c_int(i), C.c_int(B), C.c_int(Ke),
                               _ptr(r["node_tok"], C.c_int32), _ptr(r["node_S"], C.c_int64),
                               _ptr(r["node_cnt"], C.c_int32), _ptr(r["node_count"], C.c_int32),
                               _ptr(r["edge_dst"], C.c_int32), _ptr(r["edge_S"], C.c_int64),
                               _ptr(r["edge_cnt"], C.c_int32), _ptr(r["out_degree"], C.c_int32))
        return r

    # -- acceptance --------------------------------------------------------
    def accept(self, draft_tok, draft_len, sampled) -> np.ndarray:
        draft_tok = np.ascontiguousarray(draft_tok, np.int32); draft_len = np.ascontiguousarray(draft_len, np.int32)
        sampled = np.ascontiguousarray(sampled, np.int32)
        out = np.zeros(self.P, np.int32)
        self._l.orc_accept(self._h, _ptr(draft_tok, C.c_int32), _ptr(draft_len, C.c_int32),
                           _ptr(sampled, C.c_int32), _ptr(out, C.c_int32))
        return out

    def accept_commit(self, draft_tok, draft_len, sampled, sampled_logprobs, max_append):
        draft_tok = np.ascontiguousarray(draft_tok, np.int32); draft_len = np.ascontiguousarray(draft_len, np.int32)
        sampled = np.ascontiguousarray(sampled, np.int32)
        sampled_logprobs = np.ascontiguousarray(sampled_logprobs, np.float32)
        out = np.zeros(self.P, np.int32)
        st = self._l.orc_accept_commit(self._h, _ptr(draft_tok, C.c_int32), _ptr(draft_len, C.c_int32),
                                       _ptr(sampled, C.c_int32), _ptr(sampled_logprobs, C.c_float),
                                       C.c_int(max_append), _ptr(out, C.c_int32))
        return out, int(st)
