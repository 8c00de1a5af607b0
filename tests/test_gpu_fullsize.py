"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times:
the whole batch runs on the GPU, the oracle recomputes a sample of the requests one by one on the
same bytes (a full batch would take the oracle minutes)."""
import dataclasses

import pytest
import torch

from gpu_harness import Round, check_round, make_gpu, make_oracle
from paper_2609_22098_b200 import synth

pytestmark = pytest.mark.gpu


def run(wl, T, theta, reqs, seed, round_seed=77, B=None, rounds=1):
    rnd = Round(wl, seed=seed, B=B, theta=theta)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    orc = make_oracle(wl, rnd.table)
    tot = None
    for k in range(rounds):
        st = check_round(ts, orc, rnd, T, round_seed=round_seed + k, reqs=reqs)
        assert st["trees"] == len(reqs)
        tot = st if tot is None else {key: (tot[key] + st[key] if isinstance(st[key], int) else st[key]) for key in st}
    return tot


def test_serve32_full_size_every_request_three_rounds():
    wl = synth.WORKLOADS["serve32"]
    st = run(wl, 1.0, wl.theta, reqs=list(range(32)), seed=2609, rounds=3)
    assert st["nodes"] > 0 and st["trees"] == 96 and st["trees_exempt"] <= 4 and st["walks_exempt"] <= 6, st


@pytest.mark.parametrize("T", [0.0, 0.7, 1.0])
@pytest.mark.parametrize("theta", [0.3, 0.1, 0.03])
def test_decode_full_size(T, theta):
    wl = synth.WORKLOADS["decode"]
    st = run(wl, T, theta, reqs=[0], seed=31 + int(10 * T), rounds=2)
    assert st["trees"] == 2


@pytest.mark.parametrize("T", [0.7, 1.3])
def test_wide_full_size_three_requests(T):
    wl = synth.WORKLOADS["wide"]
    st = run(wl, T, wl.theta, reqs=[0, 3, 7], seed=5)
    assert st["nodes"] >= 48


def test_sweep_largest_batch_is_the_chain():
    wl = synth.WORKLOADS["sweep"]
    theta = synth.sweep_theta(128, seed=9)
    assert theta >= 1.0 and synth.sweep_theta(1, seed=9) < synth.sweep_theta(16, seed=9) < 1.0
    st = run(wl, 1.0, theta, reqs=[0, 64, 127], seed=9, B=128)
    assert st["nodes"] == 3 * wl.D          # theta >= 1: every request is a chain of D nodes


@pytest.mark.parametrize("B,reqs", [(1, [0]), (4, [0, 1, 2, 3]), (16, [1, 9]), (64, [0, 21, 42, 63])])
def test_sweep_batches(B, reqs):
    wl = synth.WORKLOADS["sweep"]
    st = run(wl, 1.0, synth.sweep_theta(B, seed=9), reqs=reqs, seed=10, B=B)
    assert st["trees"] == len(reqs)


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_paper_shape_full_size_sampled_requests(T):
    # the paper's own head and tree shape (rank 256, block of 7, 56 nodes) on the full vocabulary and batch
    wl = synth.WORKLOADS["paper"]
    st = run(wl, T, wl.theta, reqs=[0, 13, 31], seed=2610)
    assert st["trees"] == 3 and st["nodes"] > 0
