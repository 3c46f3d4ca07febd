"""ctypes binding of the fp64 CPU oracle (``moc_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the bench's
CPU-baseline leg.  The CUDA library never imports or links it.  The only code
here is argument marshalling; all arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "moc_oracle.c")
_LIB = os.path.join(_DIR, "libmoc_oracle.so")
WHOLE_SHOT = -1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the row loops) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("H", C.c_int), ("L", C.c_int), ("d", C.c_int), ("C", C.c_int), ("k", C.c_int),
                ("win_back", C.c_int), ("win_fwd", C.c_int), ("causal", C.c_int),
                ("off", C.c_void_p), ("shot", C.c_void_p), ("mod", C.c_void_p)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.moc_oracle_pair_count.restype = C.c_int64
        _lib.moc_oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return C.c_void_p(a.ctypes.data) if a is not None else C.c_void_p(0)


def philox4x32(ctr, key):
    """Philox4x32-10 of one counter block (4 x uint32) under a key (2 x uint32)."""
    c = np.ascontiguousarray(ctr, np.uint32)
    k = np.ascontiguousarray(key, np.uint32)
    out = np.zeros(4, np.uint32)
    _load().moc_oracle_philox4x32(_p(c), _p(k), _p(out))
    return out


def num_threads() -> int:
    return int(_load().moc_oracle_num_threads())


class Oracle:
    """One problem instance: shapes, chunk table, k, window, causality."""

    def __init__(self, n_heads, n_tokens, head_dim, chunk_off, chunk_shot, chunk_mod, top_k,
                 win_back=0, win_fwd=0, causal=True):
        self.off = np.ascontiguousarray(chunk_off, np.int32)
        self.shot = np.ascontiguousarray(chunk_shot, np.int32)
        self.mod = np.ascontiguousarray(chunk_mod, np.uint8)
        self.H, self.L, self.d, self.k = int(n_heads), int(n_tokens), int(head_dim), int(top_k)
        self.C = len(self.shot)
        assert len(self.off) == self.C + 1 and self.off[0] == 0 and self.off[-1] == self.L
        assert np.all(np.diff(self.off) > 0)
        self.cfg = _Cfg(self.H, self.L, self.d, self.C, self.k, int(win_back), int(win_fwd), int(bool(causal)),
                        self.off.ctypes.data, self.shot.ctypes.data, self.mod.ctypes.data)
        self.lib = _load()

    @classmethod
    def from_workload(cls, wl, n_heads=None):
        lay = wl.layout
        return cls(wl.n_heads if n_heads is None else n_heads, lay.n_tokens, wl.head_dim, lay.chunk_off,
                   lay.chunk_shot, lay.chunk_mod, wl.top_k, wl.win_back, wl.win_fwd, wl.causal)

    def _u16(self, a):
        a = np.ascontiguousarray(a)
        assert a.dtype == np.uint16 and a.shape == (self.H, self.L, self.d), (a.dtype, a.shape)
        return a

    @staticmethod
    def _rows(rows):
        rows = np.ascontiguousarray(rows, np.int32).reshape(-1, 2)
        return rows

    def all_rows(self):
        h, i = np.meshgrid(np.arange(self.H), np.arange(self.L), indexing="ij")
        return np.stack([h.ravel(), i.ravel()], 1).astype(np.int32)

    def chunk_pool(self, K):
        K = self._u16(K)
        desc = np.empty((self.H, self.C, self.d), np.float64)
        self.lib.moc_oracle_chunk_pool(C.byref(self.cfg), _p(K), _p(desc))
        return desc

    def scores(self, Q, desc, rows):
        Q, rows = self._u16(Q), self._rows(rows)
        out = np.empty((len(rows), self.C), np.float64)
        self.lib.moc_oracle_scores(C.byref(self.cfg), _p(Q), _p(desc), C.c_int(len(rows)), _p(rows), _p(out))
        return out

    def route(self, Q, desc, with_scores=False):
        Q = self._u16(Q)
        desc = np.ascontiguousarray(desc, np.float64)
        sel = np.empty((self.H, self.L, self.k), np.int32)
        ss = np.empty((self.H, self.L, self.k), np.float64) if with_scores else None
        nx = np.empty((self.H, self.L), np.float64) if with_scores else None
        self.lib.moc_oracle_route(C.byref(self.cfg), _p(Q), _p(desc), _p(sel), _p(ss), _p(nx))
        return (sel, ss, nx) if with_scores else sel

    def token_mask(self, i, sel_row):
        sel_row = np.ascontiguousarray(sel_row, np.int32)
        assert sel_row.shape == (self.k,)
        mask = np.empty(self.L, np.uint8)
        self.lib.moc_oracle_token_mask(C.byref(self.cfg), C.c_int(int(i)), _p(sel_row), _p(mask))
        return mask

    def pair_count(self, sel_idx, rows=None):
        sel_idx = np.ascontiguousarray(sel_idx, np.int32)
        rows = self.all_rows() if rows is None else self._rows(rows)
        return int(self.lib.moc_oracle_pair_count(C.byref(self.cfg), _p(sel_idx), C.c_int(len(rows)), _p(rows)))

    def attend(self, Q, K, V, sel_idx, rows=None, scale=0.0):
        """(O [n, d], lse [n]) of the listed (head, token) rows; all rows when None."""
        Q, K, V = self._u16(Q), self._u16(K), self._u16(V)
        sel_idx = np.ascontiguousarray(sel_idx, np.int32)
        assert sel_idx.shape == (self.H, self.L, self.k)
        rows = self.all_rows() if rows is None else self._rows(rows)
        O = np.empty((len(rows), self.d), np.float64)
        lse = np.empty(len(rows), np.float64)
        self.lib.moc_oracle_attend_rows(C.byref(self.cfg), _p(Q), _p(K), _p(V), _p(sel_idx), C.c_double(scale),
                                        C.c_int(len(rows)), _p(rows), _p(O), _p(lse))
        return O, lse

    def num_shots(self) -> int:
        return int(self.lib.moc_oracle_num_shots(C.byref(self.cfg)))

    def outer_route(self, Xq, Xk, q0, q1, top_m):
        """Outer-loop routing of the query block [q0, q1): (shot descriptors [H, S, d], scores [H, S],
        selected shots [H, M], -1 padded)."""
        Xq, Xk = self._u16(Xq), self._u16(Xk)
        S = self.num_shots()
        desc = np.empty((self.H, S, self.d), np.float64)
        sc = np.empty((self.H, S), np.float64)
        sel = np.empty((self.H, int(top_m)), np.int32)
        self.lib.moc_oracle_outer_route(C.byref(self.cfg), _p(Xq), _p(Xk), C.c_int(int(q0)), C.c_int(int(q1)),
                                        C.c_int(int(top_m)), _p(desc), _p(sc), _p(sel))
        return desc, sc, sel

    def context_drop(self, sel_idx, p_max, lam, seed):
        """Context drop-off / drop-in (Sec. 3.1) applied to a copy of sel_idx.  Returns
        (edited sel_idx, n_dropped, n_drawn, n_added), the last three [H, L] int32."""
        out = np.ascontiguousarray(sel_idx, np.int32).copy()
        assert out.shape == (self.H, self.L, self.k)
        nd, nm, na = (np.zeros((self.H, self.L), np.int32) for _ in range(3))
        self.lib.moc_oracle_context_drop(C.byref(self.cfg), _p(out), C.c_float(p_max), C.c_float(lam),
                                         C.c_uint64(int(seed)), _p(nd), _p(nm), _p(na))
        return out, nd, nm, na

    def attend_bwd(self, Q, K, V, dO, sel_idx, rows=None, key_head=0, key_range=None, scale=0.0):
        """dQ [n, d] of the listed rows and (dK, dV) [t1-t0, d] of tokens ``key_range`` of
        ``key_head`` (summed over every query of that head that selects them)."""
        Q, K, V, dO = self._u16(Q), self._u16(K), self._u16(V), self._u16(dO)
        sel_idx = np.ascontiguousarray(sel_idx, np.int32)
        rows = np.zeros((0, 2), np.int32) if rows is None else self._rows(rows)
        t0, t1 = (0, 0) if key_range is None else (int(key_range[0]), int(key_range[1]))
        dQ = np.empty((len(rows), self.d), np.float64)
        dK = np.empty((max(t1 - t0, 0), self.d), np.float64)
        dV = np.empty((max(t1 - t0, 0), self.d), np.float64)
        self.lib.moc_oracle_attend_bwd(C.byref(self.cfg), _p(Q), _p(K), _p(V), _p(dO), _p(sel_idx),
                                       C.c_double(scale), C.c_int(len(rows)), _p(rows), _p(dQ),
                                       C.c_int(int(key_head)), C.c_int(t0), C.c_int(t1), _p(dK), _p(dV))
        return dQ, dK, dV
