"""Seeded synthetic inputs for the TreeSpark hot path.

This module only *makes inputs*: drafter base logits ``U``, the Markov-head factors ``A`` and
``W``, anchor tokens, calibration tables, price (theta) schedules and — once a tree exists — the
target logits ``Z`` of its nodes.  It holds none of the method's arithmetic (no softmax, no top-k,
no sampling, no calibration apply, no tree logic), so both the CPU oracle's tests and the CUDA
path's tests can feed from it without sharing any of the code under test.

Everything is drawn from a counter-based Philox4x32-10 stream written here with torch integer
ops, so the same generator runs on the CPU (tests) and on the GPU (full-size bench inputs).
Transcendental functions are not bit-identical across devices, therefore a tensor is always
generated ONCE and the same bytes are handed to both sides.

The five workload recipes follow the benchmark configurations this build is measured on
(vocabulary 32,000 / 151,936 / 128,256; block depth 4 / 8 / 16; Markov rank 16 / 64 / 128; sibling
cap 4 / 8 / 16; node cap 16 / 64 / 256).  They stand in for the paper's Qwen3 + DSpark workloads
(Section 5.1), whose checkpoints and datasets are not needed here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Sequence

import torch

_M32 = 0xFFFFFFFF
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85

# Stream ids >= 16 belong to the harness; the library's own streams are 1..4.
STREAM_U = 16
STREAM_A = 17
STREAM_W = 18
STREAM_Z = 19
STREAM_MISC = 20


def _mulhilo(a: int, b: torch.Tensor):
    """32x32 -> (hi, lo) with b a non-negative int64 tensor < 2^32 and a python int < 2^32.

    The product can exceed 2^63; int64 arithmetic wraps modulo 2^64, and both halves are taken
    with masks after an arithmetic shift, which yields the right bits.
    """
    prod = b * a  # wraps mod 2^64, bits are still the low 64 bits of the true product
    lo = prod & _M32
    hi = (prod >> 32) & _M32
    return hi, lo


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Philox4x32 with 10 rounds on int64 tensors holding 32-bit words.  Returns 4 tensors."""
    k0 &= _M32
    k1 &= _M32
    for _ in range(10):
        hi0, lo0 = _mulhilo(_PHILOX_M0, c0)
        hi1, lo1 = _mulhilo(_PHILOX_M1, c2)
        n0 = hi1 ^ c1 ^ k0
        n1 = lo1
        n2 = hi0 ^ c3 ^ k1
        n3 = lo0
        c0, c1, c2, c3 = n0, n1, n2, n3
        k0 = (k0 + _PHILOX_W0) & _M32
        k1 = (k1 + _PHILOX_W1) & _M32
    return c0, c1, c2, c3


def philox_words(seed: int, stream: int, tag_lo: int, tag_hi: int, n_calls: int, device,
                 start: int = 0):
    """``n_calls`` consecutive Philox outputs, counter = (i, tag_lo, tag_hi, stream<<24)."""
    i = torch.arange(start, start + n_calls, dtype=torch.int64, device=device)
    c1 = torch.full_like(i, tag_lo & _M32)
    c2 = torch.full_like(i, tag_hi & _M32)
    c3 = torch.full_like(i, (stream & 0xFF) << 24)
    return philox4x32_10(i & _M32, c1, c2, c3, seed & _M32, (seed >> 32) & _M32)


def uniforms(seed: int, stream: int, tag: int, n: int, device="cpu") -> torch.Tensor:
    """n doubles in (0,1): (word + 0.5) / 2^32, four per Philox call."""
    calls = (n + 3) // 4
    w = philox_words(seed, stream, tag & _M32, (tag >> 32) & _M32, calls, device)
    x = torch.stack(w, dim=1).reshape(-1)[:n]
    return (x.to(torch.float64) + 0.5) * (1.0 / 4294967296.0)


def normals(seed: int, stream: int, tag: int, n: int, device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """n standard normals (float64) by Box-Muller, four per Philox call, generated in chunks."""
    out = torch.empty(n, dtype=torch.float64, device=device)
    done = 0
    while done < n:
        m = min(chunk, n - done)
        calls = (m + 3) // 4
        w0, w1, w2, w3 = philox_words(seed, stream, tag & _M32, (tag >> 32) & _M32, calls, device,
                                      start=done // 4)
        s = 1.0 / 4294967296.0
        u0 = (w0.to(torch.float64) + 0.5) * s
        u1 = (w1.to(torch.float64) + 0.5) * s
        u2 = (w2.to(torch.float64) + 0.5) * s
        u3 = (w3.to(torch.float64) + 0.5) * s
        r0 = torch.sqrt(-2.0 * torch.log(u0))
        r1 = torch.sqrt(-2.0 * torch.log(u2))
        a0 = (2.0 * math.pi) * u1
        a1 = (2.0 * math.pi) * u3
        z = torch.stack((r0 * torch.cos(a0), r0 * torch.sin(a0), r1 * torch.cos(a1), r1 * torch.sin(a1)), dim=1)
        out[done:done + m] = z.reshape(-1)[:m]
        done += m  # chunk is a multiple of 4, so call boundaries stay aligned
    return out


# --------------------------------------------------------------------------------------------
# Workload recipes
# --------------------------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and generator parameters of one benchmark configuration."""
    name: str
    B: int
    V: int
    D: int
    r: int
    K: int
    Nmax: int
    dtype: str                 # "f32" or "bf16" for U, A, W and Z
    theta: float               # default stop price (per-request array made by make_theta)
    temps: Sequence[float]
    u_std: float               # base logits ~ u_std * N(0,1)
    plant_lo: float            # planted-token bonus ~ U(plant_lo, plant_hi); 0,0 = none
    plant_hi: float
    plant_per_request: bool    # one strength per request (True) or per (request, depth)
    z_sigma: float             # target logits = drafter logits + z_sigma * N(0,1)
    calib_mode: int = 1        # 1 = per-depth 16-knot table, 0 = Platt scalars
    calib_b_lo: float = 0.6    # per-depth Platt intercept range sampled into the table
    calib_b_hi: float = 1.0

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    # Tiny reference case: everything fp32.
    "tiny": Workload("tiny", B=1, V=32000, D=4, r=16, K=4, Nmax=16, dtype="f32", theta=0.05,
                     temps=(0.0, 1.0), u_std=3.0, plant_lo=6.0, plant_hi=6.0,
                     plant_per_request=False, z_sigma=1.0),
    # Single-request decode shape.
    "decode": Workload("decode", B=1, V=151936, D=8, r=64, K=8, Nmax=64, dtype="bf16", theta=0.1,
                       temps=(0.0, 0.7, 1.0), u_std=4.0, plant_lo=5.0, plant_hi=9.0,
                       plant_per_request=False, z_sigma=0.8),
    # Batched serving.
    "serve32": Workload("serve32", B=32, V=151936, D=8, r=64, K=8, Nmax=64, dtype="bf16", theta=0.1,
                        temps=(1.0,), u_std=4.0, plant_lo=3.0, plant_hi=9.0,
                        plant_per_request=True, z_sigma=0.8),
    # Wide / deep trees on flat distributions.
    "wide": Workload("wide", B=8, V=128256, D=16, r=128, K=16, Nmax=256, dtype="bf16", theta=0.01,
                     temps=(0.7, 1.3), u_std=2.0, plant_lo=0.0, plant_hi=0.0,
                     plant_per_request=False, z_sigma=0.8, calib_b_lo=3.0, calib_b_hi=3.4),
    # Load sweep: same shape as serve32; the batch and the theta schedule vary.
    "sweep": Workload("sweep", B=16, V=151936, D=8, r=64, K=8, Nmax=64, dtype="bf16", theta=0.1,
                      temps=(1.0,), u_std=4.0, plant_lo=3.0, plant_hi=9.0,
                      plant_per_request=True, z_sigma=0.8),
    # The paper's own head and tree shape (Section 5.1: rank 256, block of 7, at most 56 nodes, 8 siblings)
    # on the serving batch; inputs as in serve32.
    "paper": Workload("paper", B=32, V=151936, D=7, r=256, K=8, Nmax=56, dtype="bf16", theta=0.1,
                      temps=(1.0,), u_std=4.0, plant_lo=3.0, plant_hi=9.0,
                      plant_per_request=True, z_sigma=0.8),
}

SWEEP_BATCHES = (1, 4, 16, 64, 128)


def sweep_theta(batch: int, seed: int) -> float:
    """Seeded monotone load->theta schedule of the load sweep: the price rises with the batch and
    reaches the chain sentinel (theta >= 1) at the largest batch."""
    base = {1: 0.05, 4: 0.08, 16: 0.15, 64: 0.4, 128: 1.0}
    vals = []
    for i, b in enumerate(SWEEP_BATCHES):
        j = float(uniforms(seed, STREAM_MISC, 0x7E7A00 + i, 1)[0])
        v = base[b] * (0.9 + 0.2 * j)
        vals.append(v if b != 128 else max(v, 1.0))
    vals = sorted(vals)
    return vals[SWEEP_BATCHES.index(batch)]


def _cast(x: torch.Tensor, wl: Workload) -> torch.Tensor:
    return x.to(wl.torch_dtype).contiguous()


def make_head(wl: Workload, seed: int, device="cpu"):
    """Markov-head factors: A [V][r] ~ N(0, 1/r), W [r][V] ~ N(0, variance 0.5)."""
    A = normals(seed, STREAM_A, 0, wl.V * wl.r, device).reshape(wl.V, wl.r) * math.sqrt(1.0 / wl.r)
    W = normals(seed, STREAM_W, 0, wl.r * wl.V, device).reshape(wl.r, wl.V) * math.sqrt(0.5)
    return _cast(A, wl), _cast(W, wl)


def make_base_logits(wl: Workload, seed: int, device="cpu", B: Optional[int] = None) -> torch.Tensor:
    """Base logits U [B][D+1][V].  Rows 0..D-1 are the drafter's per-depth logits (row d scores the
    children of a parent at depth d); row D exists only so that target logits can be synthesised
    for nodes at depth D and is never given to the library."""
    B = wl.B if B is None else B
    rows = B * (wl.D + 1)
    U = normals(seed, STREAM_U, 0, rows * wl.V, device).reshape(B, wl.D + 1, wl.V) * wl.u_std
    if wl.plant_hi > 0.0:
        pos = uniforms(seed, STREAM_MISC, 1, rows, device).reshape(B, wl.D + 1)
        tok = torch.clamp((pos * wl.V).to(torch.int64), max=wl.V - 1)
        if wl.plant_per_request:
            s = uniforms(seed, STREAM_MISC, 2, B, device).reshape(B, 1).expand(B, wl.D + 1)
        else:
            s = uniforms(seed, STREAM_MISC, 2, rows, device).reshape(B, wl.D + 1)
        bonus = wl.plant_lo + (wl.plant_hi - wl.plant_lo) * s
        U.scatter_add_(2, tok.unsqueeze(-1), bonus.unsqueeze(-1))
    return _cast(U, wl)


def make_anchor(wl: Workload, seed: int, device="cpu", B: Optional[int] = None) -> torch.Tensor:
    B = wl.B if B is None else B
    u = uniforms(seed, STREAM_MISC, 3, B, device)
    return torch.clamp((u * wl.V).to(torch.int64), max=wl.V - 1).to(torch.int32)


def make_theta(wl: Workload, B: Optional[int] = None, theta: Optional[float] = None, device="cpu") -> torch.Tensor:
    B = wl.B if B is None else B
    return torch.full((B,), wl.theta if theta is None else theta, dtype=torch.float32, device=device)


CALIB_KNOTS = 16
CALIB_LO = -10.0
CALIB_HI = 10.0


def make_calibration_table(wl: Workload, seed: int, kind: str = "fit") -> torch.Tensor:
    """Per-depth monotone table [D][16] (float32, CPU) over knots uniform in logit space on
    [CALIB_LO, CALIB_HI].  Row d is a logistic curve sampled at the knots with a seeded slope
    a_d ~ U(0.66, 0.79) (the cross-scale range of fitted slopes, Section 3.4) and intercept b_d:
    kind="platt" draws b_d ~ U(-0.6, -0.3) around the published intercept, kind="fit" draws it from
    the workload's (calib_b_lo, calib_b_hi), a range chosen so that the estimate tracks the edge
    acceptance this synthetic target actually shows."""
    ua = uniforms(seed, STREAM_MISC, 4, wl.D)
    ub = uniforms(seed, STREAM_MISC, 5, wl.D)
    a = 0.66 + (0.79 - 0.66) * ua
    if kind == "platt":
        b = -0.6 + 0.3 * ub
    elif kind == "fit":
        b = wl.calib_b_lo + (wl.calib_b_hi - wl.calib_b_lo) * ub
    else:
        raise ValueError(kind)
    t = torch.linspace(CALIB_LO, CALIB_HI, CALIB_KNOTS, dtype=torch.float64)
    y = 1.0 / (1.0 + torch.exp(-(a[:, None] * t[None, :] + b[:, None])))
    return y.to(torch.float32).contiguous()


def make_target_logits(wl: Workload, seed: int, U_full: torch.Tensor, A: torch.Tensor, W: torch.Tensor,
                       anchor: torch.Tensor, n_nodes: torch.Tensor, tok: torch.Tensor,
                       depth: torch.Tensor, node_hash: torch.Tensor, sigma: Optional[float] = None,
                       row_chunk: int = 64):
    """Target logits for every tree node of every request, ragged.

    Row layout: request b owns rows z_row_off[b] .. z_row_off[b] + n_nodes[b]; its first row is the
    root and row 1+i is node i (canonical order).  The row of a node at depth d with token x is
    U_full[b][d] + A[x] @ W + sigma * N(0,1), the noise keyed on (seed, request, path hash of the
    node) so that it does not depend on the order in which trees were built.  The contraction here
    only synthesises a target that is correlated with the drafter; it is input data, generated once
    and given unchanged to whichever implementation is under test.

    Returns (Z [rows][V] in the workload dtype, z_row_off int64 [B+1] on the same device).
    """
    dev = U_full.device
    sigma = wl.z_sigma if sigma is None else sigma
    B = U_full.shape[0]
    n_host = n_nodes.to("cpu", torch.int64)
    off = torch.zeros(B + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(n_host + 1, 0)
    total = int(off[-1])
    Z = torch.empty(total, wl.V, dtype=wl.torch_dtype, device=dev)
    # per-row (request, depth, token, hash)
    req_l, dep_l, tok_l, hash_l = [], [], [], []
    for b in range(B):
        n = int(n_host[b])
        req_l.append(torch.full((n + 1,), b, dtype=torch.int64))
        dep_l.append(torch.cat([torch.zeros(1, dtype=torch.int64), depth[b, :n].to("cpu", torch.int64)]))
        tok_l.append(torch.cat([anchor[b:b + 1].to("cpu", torch.int64), tok[b, :n].to("cpu", torch.int64)]))
        hash_l.append(node_hash[b, :n + 1].to("cpu", torch.int64))
    req_c = torch.cat(req_l)
    req = req_c.to(dev)
    dep = torch.cat(dep_l).to(dev)
    tk = torch.cat(tok_l).to(dev)
    hs = torch.cat(hash_l)
    Wf = W.to(torch.float32)
    for s in range(0, total, row_chunk):
        e = min(total, s + row_chunk)
        base = U_full[req[s:e], dep[s:e]].to(torch.float32)
        bias = A[tk[s:e]].to(torch.float32) @ Wf
        noise = torch.empty(e - s, wl.V, dtype=torch.float64, device=dev)
        for i in range(s, e):
            h = int(hs[i]) & 0xFFFFFFFFFFFFFFFF
            tag = (h ^ (int(req_c[i]) * 0x9E3779B97F4A7C15)) & 0xFFFFFFFFFFFFFFFF
            noise[i - s] = normals(seed, STREAM_Z, tag, wl.V, dev)
        Z[s:e] = (base.to(torch.float64) + bias.to(torch.float64) + sigma * noise).to(wl.torch_dtype)
    return Z, off.to(dev)
