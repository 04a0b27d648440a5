"""ctypes wrapper around the C oracle (test infrastructure only).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may use
this module.  It converts numpy arrays to the oracle's plain C arguments and
back; all arithmetic is in san_oracle.c.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_lib = None


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(C.POINTER(ty))


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_create.restype = C.c_void_p
        L.oracle_create.argtypes = [C.c_int] * 7 + [C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int), C.c_int, C.c_int]
        L.oracle_destroy.argtypes = [C.c_void_p]
        L.oracle_destroy.restype = None
        for name in ("oracle_js_divergence", "oracle_layer_js", "oracle_block_sim"):
            getattr(L, name).restype = C.c_double
        L.oracle_js_divergence.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int]
        L.oracle_layer_js.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int, C.c_int, C.c_long, C.POINTER(C.c_int)]
        L.oracle_block_sim.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_int, C.c_int]
        L.oracle_greedy_policy.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_double, C.POINTER(C.c_int)]
        L.oracle_policy_from_sizes.argtypes = [C.POINTER(C.c_int), C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.oracle_policy_from_map.argtypes = [C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.oracle_self_append.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.oracle_mem_set.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_long]
        L.oracle_beam_reorder.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.oracle_self_attend.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_float), C.POINTER(C.c_double), C.c_long, C.POINTER(C.c_double)]
        L.oracle_encdec_attend.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_float), C.POINTER(C.c_double), C.c_long, C.POINTER(C.c_double)]
        L.oracle_aan_step.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_float), C.POINTER(C.c_double)]
        L.oracle_full_block.argtypes = [C.c_int] * 5 + [C.POINTER(C.c_float)] * 3 + [C.POINTER(C.c_double)] * 2
        _lib = L
    return _lib


class OracleError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        raise OracleError(f"{what}: oracle status {rc}")


def policy_from_sizes(sizes: Sequence[int], n_layers: int) -> Tuple[np.ndarray, np.ndarray]:
    s = _i32(sizes)
    bol = np.full(n_layers, -1, np.int32)
    first = np.full(max(len(s), 1), -1, np.int32)
    rc = lib().oracle_policy_from_sizes(_p(s, C.c_int) if len(s) else None, len(s), n_layers, _p(bol, C.c_int), _p(first, C.c_int))
    _check(rc, "policy_from_sizes")
    return bol, first[:len(s)]


def policy_from_map(block_of_layer: Sequence[int]):
    m = _i32(block_of_layer)
    M = len(m)
    sizes = np.zeros(M, np.int32)
    first = np.zeros(M, np.int32)
    nb = C.c_int(0)
    rc = lib().oracle_policy_from_map(_p(m, C.c_int), M, _p(sizes, C.c_int), _p(first, C.c_int), C.byref(nb))
    _check(rc, "policy_from_map")
    return sizes[:nb.value].copy(), first[:nb.value].copy()


def js_divergence(p, q) -> float:
    p = np.ascontiguousarray(p, np.float64)
    q = np.ascontiguousarray(q, np.float64)
    return float(lib().oracle_js_divergence(_p(p, C.c_double), _p(q, C.c_double), len(p)))


def layer_js(Sa, Sb, lens) -> float:
    Sa = np.ascontiguousarray(Sa, np.float64)
    Sb = np.ascontiguousarray(Sb, np.float64)
    n, H, ld = Sa.shape
    lens = _i32(lens)
    return float(lib().oracle_layer_js(_p(Sa, C.c_double), _p(Sb, C.c_double), n, H, ld, _p(lens, C.c_int)))


def block_sim(JS, m: int, n: int) -> float:
    JS = np.ascontiguousarray(JS, np.float64)
    return float(lib().oracle_block_sim(_p(JS, C.c_double), JS.shape[0], m, n))


def greedy_policy(JS, theta: float):
    JS = np.ascontiguousarray(JS, np.float64)
    M = JS.shape[0]
    sizes = np.zeros(M, np.int32)
    nb = lib().oracle_greedy_policy(_p(JS, C.c_double), M, float(theta), _p(sizes, C.c_int))
    return [int(x) for x in sizes[:nb]]


def full_block(Q, K, V, causal: bool, want_S: bool = True):
    """Full-sequence shared attention.  Q, K: [l,H,dh]; V: [n_layers,l,H,dh]."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    l, H, dh = Q.shape
    nl = V.shape[0]
    S = np.zeros((H, l, l), np.float64) if want_S else None
    O = np.zeros((nl, l, H, dh), np.float64)
    rc = lib().oracle_full_block(l, H, dh, nl, int(causal), _p(Q, C.c_float), _p(K, C.c_float), _p(V, C.c_float),
                                 _p(S, C.c_double), _p(O, C.c_double))
    _check(rc, "full_block")
    return S, O


class Oracle:
    """State of one decode run: caches, encoder memory, one S per block."""

    def __init__(self, n_layers, n_heads, d_head, n_sent, beam, max_tgt, max_src,
                 self_sizes, encdec_sizes, encdec_shared_context=False):
        ss, es = _i32(self_sizes), _i32(encdec_sizes)
        self.M, self.H, self.dh = n_layers, n_heads, d_head
        self.n_sent, self.beam, self.n_seqs = n_sent, beam, n_sent * beam
        self.max_tgt, self.max_src = max_tgt, max_src
        self._h = lib().oracle_create(n_layers, n_heads, d_head, n_sent, beam, max_tgt, max_src,
                                      _p(ss, C.c_int), len(ss), _p(es, C.c_int), len(es),
                                      int(bool(encdec_shared_context)))
        if not self._h:
            raise OracleError("invalid sharing policy")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def self_append(self, layer, seq_ids, pos, k, v):
        seq_ids, pos = _i32(seq_ids), _i32(pos)
        k = None if k is None else _f32(k)
        v = None if v is None else _f32(v)
        _check(lib().oracle_self_append(self._h, layer, len(seq_ids), _p(seq_ids, C.c_int), _p(pos, C.c_int),
                                        _p(k, C.c_float), _p(v, C.c_float)), "self_append")

    def mem_set(self, layer, sentence, K, V):
        """K, V: [Ls, H, dh] (K may be None)."""
        V = _f32(V)
        K = None if K is None else _f32(K)
        Ls = V.shape[0]
        _check(lib().oracle_mem_set(self._h, layer, sentence, Ls, _p(K, C.c_float), _p(V, C.c_float),
                                    self.H * self.dh), "mem_set")

    def beam_reorder(self, src, lens):
        src, lens = _i32(src), _i32(lens)
        _check(lib().oracle_beam_reorder(self._h, _p(src, C.c_int), _p(lens, C.c_int)), "beam_reorder")

    def self_attend(self, layer, seq_ids, lens, q, want_S=True):
        seq_ids, lens = _i32(seq_ids), _i32(lens)
        n = len(seq_ids)
        q = None if q is None else _f32(q)
        ld = self.max_tgt
        S = np.zeros((n, self.H, ld), np.float64) if want_S else None
        O = np.zeros((n, self.H, self.dh), np.float64)
        _check(lib().oracle_self_attend(self._h, layer, n, _p(seq_ids, C.c_int), _p(lens, C.c_int), _p(q, C.c_float),
                                        _p(S, C.c_double), ld, _p(O, C.c_double)), "self_attend")
        return S, O

    def encdec_attend(self, layer, seq_ids, q, want_S=True):
        seq_ids = _i32(seq_ids)
        n = len(seq_ids)
        q = None if q is None else _f32(q)
        ld = self.max_src
        S = np.zeros((n, self.H, ld), np.float64) if want_S else None
        O = np.zeros((n, self.H, self.dh), np.float64)
        _check(lib().oracle_encdec_attend(self._h, layer, n, _p(seq_ids, C.c_int), _p(q, C.c_float),
                                          _p(S, C.c_double), ld, _p(O, C.c_double)), "encdec_attend")
        return S, O

    def aan_step(self, layer, seq_ids, t, x):
        seq_ids, t, x = _i32(seq_ids), _i32(t), _f32(x)
        out = np.zeros((len(seq_ids), self.H * self.dh), np.float64)
        _check(lib().oracle_aan_step(self._h, layer, len(seq_ids), _p(seq_ids, C.c_int), _p(t, C.c_int),
                                     _p(x, C.c_float), _p(out, C.c_double)), "aan_step")
        return out
