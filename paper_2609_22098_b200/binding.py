"""Thin ctypes binding over the TreeSpark C ABI (``include/treespark.h``).

Argument marshalling only: every step of the path runs in the library's kernels.  torch provides
device memory and the current stream.  The compiled library must exist beside this file; a missing
library is an error (there is no CPU fallback).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtreespark.so")

TS_OK = 0
DTYPE_F32, DTYPE_BF16 = 0, 1
KNOTS = 16

ABLATE_CALIB_QT = 1
TEST_FORCE_FMA, TEST_NO_TMA, TEST_NO_FEW, TEST_NO_SEED, \
    TEST_SHORT_WAITS, TEST_LOST_ARRIVAL, TEST_PERSIST, TEST_NO_UMMA, TEST_NO_TAIL = 1, 2, 4, 8, 16, 32, 64, 128, 256

EXPORTS = ("ts_create", "ts_destroy", "ts_set_ablation", "ts_set_test_mode", "ts_workspace_bytes", "ts_last_error_string",
           "ts_score_parents", "ts_score_parents_static", "ts_expand_tree", "ts_verify_tree",
           "ts_allocate_budget", "ts_calib_accumulate", "ts_calib_refit", "ts_calib_load_table",
           "ts_emit_attention_inputs", "ts_profile_enable", "ts_profile_read", "ts_kernel_name")


class TsConfig(C.Structure):
    _fields_ = [("V", C.c_int32), ("D", C.c_int32), ("r", C.c_int32), ("K", C.c_int32), ("Nmax", C.c_int32),
                ("max_batch", C.c_int32), ("dt_U", C.c_int32), ("dt_A", C.c_int32), ("dt_W", C.c_int32),
                ("dt_Z", C.c_int32), ("calib_mode", C.c_int32), ("platt_a", C.c_float), ("platt_b", C.c_float),
                ("calib_lo", C.c_float), ("calib_hi", C.c_float), ("calib_table", C.POINTER(C.c_float))]


_lib = None


def load_library() -> C.CDLL:
    """Load the compiled library; raises if it has not been built (run ``python -m paper_2609_22098_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2609_22098_b200.build.build(); "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.ts_last_error_string.restype = C.c_char_p
        L.ts_workspace_bytes.restype = C.c_size_t
        L.ts_workspace_bytes.argtypes = [C.c_void_p, C.c_int32]
        L.ts_create.argtypes = [C.POINTER(TsConfig), C.POINTER(C.c_void_p)]
        L.ts_destroy.argtypes = [C.c_void_p]
        L.ts_set_ablation.argtypes = [C.c_void_p, C.c_uint32]
        L.ts_set_ablation.restype = C.c_int32
        L.ts_set_test_mode.argtypes = [C.c_void_p, C.c_uint32]
        L.ts_set_test_mode.restype = C.c_int32
        vp, i32, f32, u64, sz = C.c_void_p, C.c_int32, C.c_float, C.c_uint64, C.c_size_t
        L.ts_score_parents.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, f32, u64] + [vp] * 6 + [vp, sz, vp]
        L.ts_score_parents_static.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, f32, u64] + [vp] * 6 + [vp]
        L.ts_expand_tree.argtypes = [vp, vp, vp, vp, i32, vp, vp, f32, u64] + [vp] * 15 + [vp, sz, vp]
        L.ts_verify_tree.argtypes = [vp, vp, vp, vp, vp, vp, i32] + [vp] * 9 + [f32, u64] + [vp] * 7 + [vp, sz, vp]
        L.ts_allocate_budget.argtypes = [vp, i32, i32] + [vp] * 14 + [vp, sz, vp]
        L.ts_calib_accumulate.argtypes = [vp, i32] + [vp] * 8 + [vp]
        L.ts_calib_refit.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
        L.ts_calib_load_table.argtypes = [vp, vp, vp]
        L.ts_emit_attention_inputs.argtypes = [vp, i32] + [vp] * 9 + [vp]
        L.ts_profile_enable.argtypes = [vp, i32]
        L.ts_profile_read.argtypes = [vp, i32, vp, vp, i32]
        L.ts_kernel_name.argtypes = [i32]
        L.ts_kernel_name.restype = C.c_char_p
        for n in ("ts_create", "ts_destroy", "ts_score_parents", "ts_score_parents_static", "ts_expand_tree", "ts_verify_tree",
                  "ts_allocate_budget", "ts_calib_accumulate", "ts_calib_refit", "ts_calib_load_table",
           "ts_emit_attention_inputs", "ts_profile_enable", "ts_profile_read"):
            getattr(L, n).restype = C.c_int32
        _lib = L
    return _lib


class TreeSparkError(RuntimeError):
    pass


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class TreeSpark:
    """A library context for one configuration plus its caller-owned workspace."""

    def __init__(self, V, D, r, K, Nmax, max_batch, dtype=torch.bfloat16, calib_mode=0, platt_a=0.67,
                 platt_b=-0.46, calib_lo=-10.0, calib_hi=10.0, calib_table=None, device="cuda", test_mode=0):
        self.lib = load_library()
        self.V, self.D, self.r, self.K, self.Nmax, self.max_batch = V, D, r, K, Nmax, max_batch
        self.dtype = dtype
        self.device = torch.device(device)
        self.words = (Nmax + 63) // 64
        dt = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_F32
        table_arr = None
        if calib_mode == 1:
            flat = [float(x) for x in torch.as_tensor(calib_table, dtype=torch.float32).reshape(-1).tolist()]
            assert len(flat) == D * KNOTS
            table_arr = (C.c_float * len(flat))(*flat)
        cfg = TsConfig(V, D, r, K, Nmax, max_batch, dt, dt, dt, dt, calib_mode, platt_a, platt_b, calib_lo, calib_hi,
                       C.cast(table_arr, C.POINTER(C.c_float)) if table_arr is not None else None)
        self._ctx = C.c_void_p()
        with torch.cuda.device(self.device):
            self._check(self.lib.ts_create(C.byref(cfg), C.byref(self._ctx)))
            if test_mode:   # the library's own tests: other kernel paths, shortened waits
                self._check(self.lib.ts_set_test_mode(self._ctx, int(test_mode)))
        self.ws_bytes = int(self.lib.ts_workspace_bytes(self._ctx, max_batch))
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device)

    def close(self):
        if getattr(self, "_ctx", None):
            self.lib.ts_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, code: int):
        if code != TS_OK:
            raise TreeSparkError(f"status {code}: {self.lib.ts_last_error_string().decode()}")

    def set_test_mode(self, flags: int):
        """Switch test modes after construction; only the modes that leave the workspace size alone
        (wait limits, lost arrival, seeding) may be changed this way."""
        self._check(self.lib.ts_set_test_mode(self._ctx, int(flags)))

    def set_ablation(self, flags: int):
        self._check(self.lib.ts_set_ablation(self._ctx, int(flags)))

    # -- instrumentation ---------------------------------------------------------------------------
    def profile_enable(self, capacity: int):
        self._check(self.lib.ts_profile_enable(self._ctx, int(capacity)))

    def profile_read(self, reset: bool = True):
        """{kernel name: (milliseconds, launches)} since the last reset; synchronises with the device."""
        n = 0
        while self.lib.ts_kernel_name(n) is not None:
            n += 1
        ms = (C.c_double * n)()
        cnt = (C.c_int64 * n)()
        self._check(self.lib.ts_profile_read(self._ctx, n, ms, cnt, 1 if reset else 0))
        return {self.lib.ts_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

    # -- output buffers (caller-owned; allocate once, reuse across rounds) -------------------------
    def alloc_score_outputs(self, P: int) -> Dict[str, torch.Tensor]:
        d, K = self.device, self.K
        return dict(lse0=torch.empty(P, dtype=torch.float32, device=d), lseT=torch.empty(P, dtype=torch.float32, device=d),
                    top_tok=torch.empty(P, K, dtype=torch.int32, device=d), top_logit=torch.empty(P, K, dtype=torch.float32, device=d),
                    draw_tok=torch.empty(P, K, dtype=torch.int32, device=d), draw_logit=torch.empty(P, K, dtype=torch.float32, device=d))

    def alloc_tree(self, B: int) -> Dict[str, torch.Tensor]:
        d, N = self.device, self.Nmax
        i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device=d)
        f32 = lambda *s: torch.zeros(*s, dtype=torch.float32, device=d)
        return dict(n_nodes=i32(B), tok=i32(B, N), parent=i32(B, N), depth=i32(B, N), sib_rank=i32(B, N),
                    logS=f32(B, N), q0=f32(B, N), logqT=f32(B, N), logkey=f32(B, N), pop_rank=i32(B, N),
                    node_hash=torch.zeros(B, N + 1, dtype=torch.int64, device=d), node_lseT=f32(B, N + 1),
                    mask=torch.zeros(B, N, self.words, dtype=torch.int64, device=d), n_scored=i32(B), status=i32(B))

    def alloc_verdict(self, B: int) -> Dict[str, torch.Tensor]:
        d = self.device
        i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device=d)
        return dict(acc_len=i32(B), acc_node=i32(B, self.D), acc_tok=i32(B, self.D), bonus_tok=i32(B),
                    edge_stat=torch.zeros(B, self.Nmax, dtype=torch.float32, device=d), flags=i32(B), status=i32(B))

    # -- the three calls -------------------------------------------------------------------------
    def score_parents(self, U, A, W, parent_req, parent_depth, parent_token, parent_hash, T, seed, out=None):
        P = int(parent_req.numel())
        out = out or self.alloc_score_outputs(P)
        self._check(self.lib.ts_score_parents(self._ctx, _ptr(U), _ptr(A), _ptr(W), P, _ptr(parent_req),
                                              _ptr(parent_depth), _ptr(parent_token), _ptr(parent_hash),
                                              float(T), int(seed), _ptr(out["lse0"]), _ptr(out["lseT"]),
                                              _ptr(out["top_tok"]), _ptr(out["top_logit"]), _ptr(out["draw_tok"]),
                                              _ptr(out["draw_logit"]), _ptr(self.ws), self.ws_bytes, _stream()))
        return out

    def score_parents_static(self, U, A, W, parent_req, parent_depth, parent_token, parent_hash, T, seed, out):
        """ts_score_parents for callers without a workspace: scratch is the library's built-in 8 MiB
        device array, so ``out`` must be given (nothing is allocated here either) and the number of
        parents is bounded; see the header for the sharing rules."""
        P = int(parent_req.numel())
        self._check(self.lib.ts_score_parents_static(self._ctx, _ptr(U), _ptr(A), _ptr(W), P, _ptr(parent_req),
                                                     _ptr(parent_depth), _ptr(parent_token), _ptr(parent_hash),
                                                     float(T), int(seed), _ptr(out["lse0"]), _ptr(out["lseT"]),
                                                     _ptr(out["top_tok"]), _ptr(out["top_logit"]),
                                                     _ptr(out["draw_tok"]), _ptr(out["draw_logit"]), _stream()))
        return out

    def expand_tree(self, U, A, W, anchor_tok, theta, T, seed, out=None):
        B = int(anchor_tok.numel())
        t = out or self.alloc_tree(B)
        self._check(self.lib.ts_expand_tree(self._ctx, _ptr(U), _ptr(A), _ptr(W), B, _ptr(anchor_tok), _ptr(theta),
                                            float(T), int(seed), _ptr(t["n_nodes"]), _ptr(t["tok"]), _ptr(t["parent"]),
                                            _ptr(t["depth"]), _ptr(t["sib_rank"]), _ptr(t["logS"]), _ptr(t["q0"]),
                                            _ptr(t["logqT"]), _ptr(t["logkey"]), _ptr(t["pop_rank"]),
                                            _ptr(t["node_hash"]), _ptr(t["node_lseT"]), _ptr(t["mask"]),
                                            _ptr(t["n_scored"]), _ptr(t["status"]), _ptr(self.ws), self.ws_bytes,
                                            _stream()))
        return t

    def allocate_budget(self, tree, budget, log_price=None):
        """Cut the trees of ``tree`` (the dict ts_expand_tree filled) back, in place, to ``budget`` nodes
        for the whole batch; ``log_price`` is an optional float32 device tensor of one element."""
        B = int(tree["n_nodes"].numel())
        self._check(self.lib.ts_allocate_budget(self._ctx, B, int(budget), _ptr(tree["n_nodes"]), _ptr(tree["tok"]),
                                                _ptr(tree["parent"]), _ptr(tree["depth"]), _ptr(tree["sib_rank"]),
                                                _ptr(tree["logS"]), _ptr(tree["q0"]), _ptr(tree["logqT"]),
                                                _ptr(tree["logkey"]), _ptr(tree["pop_rank"]), _ptr(tree["node_hash"]),
                                                _ptr(tree["node_lseT"]), _ptr(tree["mask"]), _ptr(log_price),
                                                _ptr(self.ws), self.ws_bytes, _stream()))
        return tree

    def emit_attention_inputs(self, anchor_tok, tree, base_pos=None, out=None):
        """Token ids, position ids and the dense additive mask of the flattened trees (Section 3.2 item 3)."""
        B, R, d = int(anchor_tok.numel()), self.Nmax + 1, self.device
        out = out or dict(flat_tok=torch.empty(B, R, dtype=torch.int32, device=d),
                          pos_ids=torch.empty(B, R, dtype=torch.int32, device=d),
                          dense_mask=torch.empty(B, R, R, dtype=torch.float32, device=d))
        self._check(self.lib.ts_emit_attention_inputs(self._ctx, B, _ptr(anchor_tok), _ptr(base_pos), _ptr(tree["n_nodes"]),
                                                      _ptr(tree["tok"]), _ptr(tree["depth"]), _ptr(tree["mask"]),
                                                      _ptr(out.get("flat_tok")), _ptr(out.get("pos_ids")),
                                                      _ptr(out.get("dense_mask")), _stream()))
        return out

    # -- calibration statistics (Section 3.4) -------------------------------------------------------
    def calib_new_stats(self) -> torch.Tensor:
        """Zeroed statistics array [2][D][16][3] (int64 holding the library's unsigned 64-bit sums)."""
        return torch.zeros(2, self.D, KNOTS, 3, dtype=torch.int64, device=self.device)

    def calib_accumulate(self, tree, verdict, stats):
        B = int(tree["n_nodes"].numel())
        self._check(self.lib.ts_calib_accumulate(self._ctx, B, _ptr(tree["n_nodes"]), _ptr(tree["parent"]),
                                                 _ptr(tree["depth"]), _ptr(tree["q0"]), _ptr(verdict["acc_len"]),
                                                 _ptr(verdict["acc_node"]), _ptr(verdict["edge_stat"]), _ptr(stats),
                                                 _stream()))
        return stats

    def calib_refit(self, stats, population=1, min_count=1, fallback=None, table=None, platt=None):
        """(table float32 [D][16], platt float64 [4] = a, b, Newton steps, edges used), both on the device."""
        table = torch.empty(self.D, KNOTS, dtype=torch.float32, device=self.device) if table is None else table
        platt = torch.empty(4, dtype=torch.float64, device=self.device) if platt is None else platt
        self._check(self.lib.ts_calib_refit(self._ctx, _ptr(stats), int(population), int(min_count), _ptr(fallback),
                                            _ptr(table), _ptr(platt), _stream()))
        return table, platt

    def calib_load_table(self, table):
        self._check(self.lib.ts_calib_load_table(self._ctx, _ptr(table), _stream()))

    def verify_tree(self, U, A, W, Z, z_row_off, anchor_tok, tree, T, seed, out=None, edge_stat=True):
        B = int(anchor_tok.numel())
        v = out or self.alloc_verdict(B)
        self._check(self.lib.ts_verify_tree(self._ctx, _ptr(U), _ptr(A), _ptr(W), _ptr(Z), _ptr(z_row_off), B,
                                            _ptr(anchor_tok), _ptr(tree["n_nodes"]), _ptr(tree["tok"]),
                                            _ptr(tree["parent"]), _ptr(tree["depth"]), _ptr(tree["sib_rank"]),
                                            _ptr(tree["node_hash"]), _ptr(tree["logqT"]), _ptr(tree["node_lseT"]),
                                            float(T), int(seed), _ptr(v["acc_len"]), _ptr(v["acc_node"]),
                                            _ptr(v["acc_tok"]), _ptr(v["bonus_tok"]),
                                            _ptr(v["edge_stat"]) if edge_stat else None, _ptr(v["flags"]),
                                            _ptr(v["status"]), _ptr(self.ws), self.ws_bytes, _stream()))
        return v


def ts_score_parents(ctx: TreeSpark, *args, **kw):
    return ctx.score_parents(*args, **kw)


def ts_expand_tree(ctx: TreeSpark, *args, **kw):
    return ctx.expand_tree(*args, **kw)


def ts_verify_tree(ctx: TreeSpark, *args, **kw):
    return ctx.verify_tree(*args, **kw)


class HostRound:
    """One whole round for callers whose buffers live in host memory.

    ``run`` copies the step's inputs (base logits, anchors, prices, target logits and their row
    offsets) from pinned host tensors to device staging buffers, runs ts_expand_tree and
    ts_verify_tree, copies the tree and the verdict back into pinned host tensors and waits for
    them.  All staging memory is allocated once in the constructor.

    ``submit`` / ``collect`` are the same round split in two for callers that keep the copy engine busy:
    ``submit`` queues the host-to-device copies of a step on a copy stream and the round behind them on the
    caller's stream, into one of two staging slots; ``collect`` waits for the oldest submitted step and
    returns its host outputs.  With two steps in flight the copies of one step run beside the kernels of
    the step before."""

    TREE_OUT = ("n_nodes", "tok", "parent", "depth", "mask")
    RESULT_KEYS = ("acc_len", "acc_tok", "bonus_tok")

    @staticmethod
    def pin_inputs(U, anchor, theta, Z, zoff):
        return {k: t.detach().to("cpu").contiguous().pin_memory()
                for k, t in dict(U=U, anchor=anchor, theta=theta, Z=Z, zoff=zoff).items()}

    def __init__(self, ts: TreeSpark, B: int, max_rows: int):
        self.ts, self.B = ts, B
        d = ts.device
        self.U = torch.empty(B, ts.D, ts.V, dtype=ts.dtype, device=d)
        self.anchor = torch.empty(B, dtype=torch.int32, device=d)
        self.theta = torch.empty(B, dtype=torch.float32, device=d)
        self.Z = torch.empty(max_rows, ts.V, dtype=ts.dtype, device=d)
        self.zoff = torch.empty(B + 1, dtype=torch.int64, device=d)
        self.tree = ts.alloc_tree(B)
        self.verdict = ts.alloc_verdict(B)
        self.host_out = {k: torch.empty_like(self.tree[k], device="cpu").pin_memory() for k in self.TREE_OUT}
        self.host_out.update({k: torch.empty_like(self.verdict[k], device="cpu").pin_memory() for k in self.RESULT_KEYS})
        self.h2d_bytes = 0
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.host_out.values())
        self._max_rows = max_rows
        self._slots = None      # second staging slot, copy stream and events: built on the first submit
        self._pending = []

    def _make_slots(self):
        ts, B, d = self.ts, self.B, self.ts.device
        slots = [dict(U=self.U, anchor=self.anchor, theta=self.theta, Z=self.Z, zoff=self.zoff, tree=self.tree,
                      verdict=self.verdict, out=self.host_out)]
        slots.append(dict(U=torch.empty_like(self.U), anchor=torch.empty_like(self.anchor), theta=torch.empty_like(self.theta),
                          Z=torch.empty_like(self.Z), zoff=torch.empty_like(self.zoff), tree=ts.alloc_tree(B),
                          verdict=ts.alloc_verdict(B),
                          out={k: torch.empty_like(v).pin_memory() for k, v in self.host_out.items()}))
        for sl in slots:
            sl["copied"] = torch.cuda.Event()
            sl["done"] = torch.cuda.Event()
            sl["free"] = torch.cuda.Event()
            sl["free"].record()
        self._copy_stream = torch.cuda.Stream(device=d)
        self._slots, self._next = slots, 0

    def submit(self, host, A, W, T, seed, edge_stat=True):
        """Queue one round; at most two may be in flight (collect the older one first)."""
        if self._slots is None:
            self._make_slots()
        if len(self._pending) >= 2:
            raise RuntimeError("HostRound.submit: two rounds already in flight; call collect() first")
        ts = self.ts
        sl = self._slots[self._next]
        self._next ^= 1
        rows = host["Z"].shape[0]
        main = torch.cuda.current_stream()
        with torch.cuda.stream(self._copy_stream):
            self._copy_stream.wait_event(sl["free"])      # the round that used this slot last has finished
            sl["U"].copy_(host["U"], non_blocking=True)
            sl["anchor"].copy_(host["anchor"], non_blocking=True)
            sl["theta"].copy_(host["theta"], non_blocking=True)
            sl["Z"][:rows].copy_(host["Z"], non_blocking=True)
            sl["zoff"].copy_(host["zoff"], non_blocking=True)
            sl["copied"].record()
        main.wait_event(sl["copied"])
        ts.expand_tree(sl["U"], A, W, sl["anchor"], sl["theta"], T, seed, out=sl["tree"])
        ts.verify_tree(sl["U"], A, W, sl["Z"], sl["zoff"], sl["anchor"], sl["tree"], T, seed, out=sl["verdict"],
                       edge_stat=edge_stat)
        for k in self.TREE_OUT:
            sl["out"][k].copy_(sl["tree"][k], non_blocking=True)
        for k in self.RESULT_KEYS:
            sl["out"][k].copy_(sl["verdict"][k], non_blocking=True)
        sl["done"].record()
        sl["free"].record()
        self._pending.append(sl)
        self.h2d_bytes = sum(host[k].numel() * host[k].element_size() for k in ("U", "anchor", "theta", "Z", "zoff"))

    def collect(self):
        """Host outputs of the oldest submitted round (waits for it)."""
        sl = self._pending.pop(0)
        sl["done"].synchronize()
        return sl["out"]

    def run(self, host, A, W, T, seed, edge_stat=True):
        ts = self.ts
        rows = host["Z"].shape[0]
        self.U.copy_(host["U"], non_blocking=True)
        self.anchor.copy_(host["anchor"], non_blocking=True)
        self.theta.copy_(host["theta"], non_blocking=True)
        ts.expand_tree(self.U, A, W, self.anchor, self.theta, T, seed, out=self.tree)
        self.Z[:rows].copy_(host["Z"], non_blocking=True)
        self.zoff.copy_(host["zoff"], non_blocking=True)
        ts.verify_tree(self.U, A, W, self.Z, self.zoff, self.anchor, self.tree, T, seed, out=self.verdict,
                       edge_stat=edge_stat)
        for k in self.TREE_OUT:
            self.host_out[k].copy_(self.tree[k], non_blocking=True)
        for k in self.RESULT_KEYS:
            self.host_out[k].copy_(self.verdict[k], non_blocking=True)
        torch.cuda.current_stream().synchronize()
        self.h2d_bytes = sum(host[k].numel() * host[k].element_size() for k in ("U", "anchor", "theta", "Z", "zoff"))
        return self.host_out
