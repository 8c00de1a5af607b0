"""ctypes access to the TreeSpark CPU oracle -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package; the
product path never does.  The oracle itself is the C file beside this one; nothing here adds
arithmetic, it only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "treespark_oracle.c")
_LIB = os.path.join(_HERE, "libtreespark_oracle.so")

KMAX = 16
DMAX = 16
KNOTS = 16

FLAG_NEAR_TOPK = 1
FLAG_NEAR_THETA = 2
FLAG_NEAR_CAP = 4
FLAG_NEAR_ACCEPT = 8
FLAG_NEAR_CDF = 16
FLAG_SATURATED = 32
FLAG_ZERO_MASS = 64
TOPK_MARGIN = 4e-6


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) if the shared object is missing or stale."""
    hdr = os.path.join(_HERE, "treespark_oracle.h")
    stale = (not os.path.exists(_LIB)) or any(os.path.getmtime(_LIB) < os.path.getmtime(f) for f in (_SRC, hdr))
    if force or stale:
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Config(C.Structure):
    _fields_ = [("V", C.c_int32), ("D", C.c_int32), ("r", C.c_int32), ("K", C.c_int32), ("Nmax", C.c_int32),
                ("calib_mode", C.c_int32), ("platt_a", C.c_double), ("platt_b", C.c_double),
                ("calib_lo", C.c_double), ("calib_hi", C.c_double), ("calib_table", C.POINTER(C.c_double)),
                ("calib_input", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.orc_path_hash.restype = C.c_uint64
        L.orc_path_hash.argtypes = [C.c_uint64, C.c_int32]
        for name in ("orc_u_gumbel", "orc_u_accept"):
            getattr(L, name).restype = C.c_double
            getattr(L, name).argtypes = [C.c_uint64, C.c_int32, C.c_uint64, C.c_int32]
        L.orc_u_bonus.restype = C.c_double
        L.orc_u_bonus.argtypes = [C.c_uint64, C.c_int32, C.c_uint64]
        L.orc_calib.restype = C.c_double
        L.orc_calib.argtypes = [C.POINTER(_Config), C.c_int32, C.c_double]
        L.orc_expand_tree.restype = C.c_int32
        _lib = L
    return _lib


def _f32(x) -> np.ndarray:
    """Exact float32 view of an input tensor/array (bf16 values are exactly representable)."""
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").float().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


class Oracle:
    """One configuration of the method (vocabulary, depth, rank, caps, calibration)."""

    def __init__(self, V, D, r, K, Nmax, calib_mode=0, platt_a=0.67, platt_b=-0.46,
                 calib_lo=-10.0, calib_hi=10.0, calib_table=None, calib_input=0):
        assert K <= KMAX and D <= DMAX
        self.V, self.D, self.r, self.K, self.Nmax = V, D, r, K, Nmax
        self.words = (Nmax + 63) // 64
        self._table = None
        if calib_mode == 1:
            self._table = np.ascontiguousarray(np.asarray(calib_table, dtype=np.float64).reshape(D, KNOTS))
        self.cfg = _Config(V, D, r, K, Nmax, calib_mode, platt_a, platt_b, calib_lo, calib_hi,
                           _p(self._table, C.c_double) if self._table is not None else None, calib_input)

    # -- scalars ---------------------------------------------------------------------------
    def calib(self, d: int, t: float) -> float:
        return lib().orc_calib(C.byref(self.cfg), d, t)

    # -- scoring ---------------------------------------------------------------------------
    def logits(self, U_row, a_row, W) -> np.ndarray:
        U_row, a_row, W = _f32(U_row), _f32(a_row), _f32(W)
        out = np.empty(self.V, dtype=np.float64)
        lib().orc_logits(C.byref(self.cfg), _p(U_row, C.c_float), _p(a_row, C.c_float), _p(W, C.c_float),
                         _p(out, C.c_double))
        return out

    def score_parent(self, U_row, a_row, W, T, seed, req, node_hash):
        U_row, a_row, W = _f32(U_row), _f32(a_row), _f32(W)
        K = self.K
        lse0, lseT = C.c_double(), C.c_double()
        top_tok = np.empty(K, np.int32); top_logit = np.empty(K, np.float64)
        draw_tok = np.empty(K, np.int32); draw_logit = np.empty(K, np.float64)
        draw_key = np.empty(K, np.float64); margins = np.empty(2 * K, np.float64)
        lib().orc_score_parent(C.byref(self.cfg), _p(U_row, C.c_float), _p(a_row, C.c_float), _p(W, C.c_float),
                               C.c_double(T), C.c_uint64(seed), C.c_int32(req), C.c_uint64(node_hash),
                               C.byref(lse0), C.byref(lseT), _p(top_tok, C.c_int32), _p(top_logit, C.c_double),
                               _p(draw_tok, C.c_int32), _p(draw_logit, C.c_double), _p(draw_key, C.c_double),
                               _p(margins, C.c_double))
        return dict(lse0=lse0.value, lseT=lseT.value, top_tok=top_tok, top_logit=top_logit,
                    draw_tok=draw_tok, draw_logit=draw_logit, draw_key=draw_key,
                    margins=np.array([margins[:K].min(), margins[K:].min()]), gaps=margins)

    # -- expansion -------------------------------------------------------------------------
    def expand_tree(self, U_req, A, W, anchor_tok, theta, T, seed, req):
        """Algorithm 1 for one request; U_req is [>=D][V] (only the first D rows are read)."""
        U_req, A, W = _f32(U_req), _f32(A), _f32(W)
        N, words = self.Nmax, self.words
        o = dict(tok=np.full(N, -1, np.int32), parent=np.full(N, -1, np.int32), depth=np.zeros(N, np.int32),
                 sib_rank=np.zeros(N, np.int32), logS=np.zeros(N, np.float64), q0=np.zeros(N, np.float64),
                 logqT=np.zeros(N, np.float64), logkey=np.zeros(N, np.float64), pop_rank=np.zeros(N, np.int32),
                 node_hash=np.zeros(N + 1, np.uint64), mask=np.zeros((N, words), np.uint64))
        n_scored, flags = C.c_int32(), C.c_uint32()
        n = lib().orc_expand_tree(C.byref(self.cfg), _p(U_req, C.c_float), _p(A, C.c_float), _p(W, C.c_float),
                                  C.c_int32(int(anchor_tok)), C.c_double(theta), C.c_double(T), C.c_uint64(seed),
                                  C.c_int32(req), _p(o["tok"], C.c_int32), _p(o["parent"], C.c_int32),
                                  _p(o["depth"], C.c_int32), _p(o["sib_rank"], C.c_int32), _p(o["logS"], C.c_double),
                                  _p(o["q0"], C.c_double), _p(o["logqT"], C.c_double), _p(o["logkey"], C.c_double),
                                  _p(o["pop_rank"], C.c_int32), _p(o["node_hash"], C.c_uint64),
                                  _p(o["mask"], C.c_uint64), C.byref(n_scored), C.byref(flags))
        o["n"] = n
        o["n_scored"] = n_scored.value
        o["flags"] = flags.value
        return o

    # -- verification ----------------------------------------------------------------------
    def verify_tree(self, U_req, A, W, Z, anchor_tok, tree, T, seed, req, closed_form=False,
                    accept_margin=1e-6, want_edge_stat=False):
        U_req, A, W, Z = _f32(U_req), _f32(A), _f32(W), _f32(Z)
        n = int(tree["n"])
        assert Z.shape[0] >= n + 1
        acc_len, bonus, flags = C.c_int32(), C.c_int32(), C.c_uint32()
        acc_node = np.full(max(self.D, 1), -1, np.int32); acc_tok = np.full(max(self.D, 1), -1, np.int32)
        edge = np.zeros(max(n, 1), np.float64) if want_edge_stat else None
        tk = np.ascontiguousarray(tree["tok"], np.int32); pa = np.ascontiguousarray(tree["parent"], np.int32)
        de = np.ascontiguousarray(tree["depth"], np.int32); sr = np.ascontiguousarray(tree["sib_rank"], np.int32)
        nh = np.ascontiguousarray(tree["node_hash"], np.uint64)
        lib().orc_verify_tree(C.byref(self.cfg), _p(U_req, C.c_float), _p(A, C.c_float), _p(W, C.c_float),
                              _p(Z, C.c_float), C.c_int32(int(anchor_tok)), C.c_int32(n), _p(tk, C.c_int32),
                              _p(pa, C.c_int32), _p(de, C.c_int32), _p(sr, C.c_int32), _p(nh, C.c_uint64),
                              C.c_double(T), C.c_uint64(seed), C.c_int32(req), C.c_int32(1 if closed_form else 0),
                              C.c_double(accept_margin), C.byref(acc_len), _p(acc_node, C.c_int32),
                              _p(acc_tok, C.c_int32), C.byref(bonus),
                              _p(edge, C.c_double) if edge is not None else None, C.byref(flags))
        return dict(acc_len=acc_len.value, acc_node=acc_node, acc_tok=acc_tok, bonus=bonus.value,
                    edge_stat=edge, flags=flags.value)

    # -- test support ----------------------------------------------------------------------
    def lossless_trials(self, U_req, A, W, Z_path, anchor_tok, theta, T, seed0, trials, mode=0, closed_form=False):
        U_req, A, W, Z_path = _f32(U_req), _f32(A), _f32(W), _f32(Z_path)
        V = self.V
        h1 = np.zeros(V, np.int64); h2 = np.zeros((V, V), np.int64)
        mn, ma = C.c_double(), C.c_double()
        lib().orc_lossless_trials(C.byref(self.cfg), _p(U_req, C.c_float), _p(A, C.c_float), _p(W, C.c_float),
                                  _p(Z_path, C.c_float), C.c_int32(int(anchor_tok)), C.c_double(theta), C.c_double(T),
                                  C.c_uint64(seed0), C.c_int64(trials), C.c_int32(mode),
                                  C.c_int32(1 if closed_form else 0), _p(h1, C.c_int64), _p(h2, C.c_int64),
                                  C.byref(mn), C.byref(ma))
        return h1, h2, mn.value, ma.value

    def draw_order_trials(self, U_row, a_row, W, T, seed0, trials):
        U_row, a_row, W = _f32(U_row), _f32(a_row), _f32(W)
        hist = np.zeros(self.V ** self.K, np.int64)
        lib().orc_draw_order_trials(C.byref(self.cfg), _p(U_row, C.c_float), _p(a_row, C.c_float), _p(W, C.c_float),
                                    C.c_double(T), C.c_uint64(seed0), C.c_int64(trials), _p(hist, C.c_int64))
        return hist.reshape((self.V,) * self.K)


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr); k = (C.c_uint32 * 2)(*key); o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def path_hash(parent_hash: int, token: int) -> int:
    return int(lib().orc_path_hash(C.c_uint64(parent_hash), C.c_int32(token)))


def u_gumbel(seed, req, node_hash, v) -> float:
    return lib().orc_u_gumbel(C.c_uint64(seed), C.c_int32(req), C.c_uint64(node_hash), C.c_int32(v))


def u_accept(seed, req, node_hash, j) -> float:
    return lib().orc_u_accept(C.c_uint64(seed), C.c_int32(req), C.c_uint64(node_hash), C.c_int32(j))


def u_bonus(seed, req, node_hash) -> float:
    return lib().orc_u_bonus(C.c_uint64(seed), C.c_int32(req), C.c_uint64(node_hash))


def run_batch(fn, items, threads: Optional[int] = None):
    """Map ``fn`` over per-request work items on a thread pool (ctypes releases the GIL)."""
    threads = threads or min(len(items), os.cpu_count() or 1)
    if threads <= 1:
        return [fn(it) for it in items], 1
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(fn, items)), threads
