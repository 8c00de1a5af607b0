"""GPU parity of the calibration-statistics calls (Section 3.4) against the CPU oracle.  Counts and
label sums are integers and compared exactly; the logit sums, the fitted scalars and the table are
floating point and compared under stated tolerances."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from oracle import calibrate as cal
from gpu_harness import Round, check_round, make_gpu, make_oracle, to_cpu
from paper_2609_22098_b200 import synth
from paper_2609_22098_b200.binding import TreeSparkError

pytestmark = pytest.mark.gpu

LO, HI = -10.0, 10.0


def small(name, **kw):
    return dataclasses.replace(synth.WORKLOADS[name], **kw)


def gpu_rounds(ts, rnd, T, seeds, stats_dev, theta=0.01):
    """Run rounds on the GPU, accumulate on the GPU, and return what the oracle needs to do the same."""
    rnd.theta.fill_(theta)
    out = []
    for s in seeds:
        tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, s)
        Z, off = rnd.target_logits(tree)
        verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, s)
        ts.calib_accumulate(tree, verdict, stats_dev)
        torch.cuda.synchronize()
        assert (tree["status"] == 0).all() and (verdict["status"] == 0).all()
        out.append((to_cpu(tree), to_cpu(verdict)))
    return out


def oracle_stats(D, rounds):
    stats = cal.new_stats(D)
    near = 0
    for g, v in rounds:
        for b in range(g["n_nodes"].numel()):
            near += cal.accumulate(stats, D, LO, HI, int(g["n_nodes"][b]), g["parent"][b].numpy(), g["depth"][b].numpy(),
                                   g["q0"][b].numpy(), v["edge_stat"][b].numpy(), int(v["acc_len"][b]),
                                   v["acc_node"][b].numpy())
    return stats, near


@pytest.mark.parametrize("name,kw,T", [
    ("serve32", dict(V=12000 + 8, B=32), 0.0),
    ("serve32", dict(V=12000 + 8, B=32), 1.0),
    ("wide", dict(V=9000, B=8), 0.7),
    ("decode", dict(V=8000), 1.0),
])
def test_accumulated_statistics_match_oracle(name, kw, T):
    wl = small(name, **kw)
    rnd = Round(wl, seed=61)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    stats_dev = ts.calib_new_stats()
    rounds = gpu_rounds(ts, rnd, T, seeds=[5, 6, 7], stats_dev=stats_dev)
    got = stats_dev.cpu().numpy()
    want, near = oracle_stats(wl.D, rounds)
    edges = sum(int(g["n_nodes"].sum()) for g, _ in rounds)
    assert edges > 3 * rnd.B and got[0, ..., 0].sum() == edges
    assert near == 0                                          # no bin decision within 1e-9 of a boundary
    assert np.array_equal(got[..., 0], want[..., 0])          # counts
    assert np.array_equal(got[..., 1], want[..., 1])          # label sums, units of 2^-24
    # logit sums: the logarithm may differ in the last place between the two sides, one unit of 2^-24
    # per edge at most
    assert (np.abs(got[..., 2] - want[..., 2]) <= want[..., 0]).all()
    if T == 0.0:
        acc = sum(int(v["acc_len"].sum()) for _, v in rounds)
        assert got[1, ..., 1].sum() == acc << 24              # committed nodes = ancestors-accepted edges labelled 1


@pytest.mark.parametrize("population,min_count,T", [(1, 1, 0.0), (1, 8, 0.0), (0, 3, 0.0), (1, 4, 1.0)])
def test_refit_matches_oracle(population, min_count, T):
    wl = small("serve32", V=12000 + 8, B=32)
    rnd = Round(wl, seed=67)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    stats_dev = ts.calib_new_stats()
    gpu_rounds(ts, rnd, T, seeds=[11, 12, 13, 14], stats_dev=stats_dev)
    stats = stats_dev.cpu().numpy()
    table_dev, platt_dev = ts.calib_refit(stats_dev, population=population, min_count=min_count)
    torch.cuda.synchronize()
    table, platt = table_dev.cpu().numpy(), platt_dev.cpu().numpy()
    a, b, it = cal.fit_platt(cal.cells_of(stats, population))
    assert platt[0] == pytest.approx(a, rel=1e-8, abs=1e-9) and platt[1] == pytest.approx(b, rel=1e-8, abs=1e-9)
    # the number of Newton steps is no parity quantity: near the optimum the last-place differences of the logarithm
    # decide when the step-halving stops; both sides must have converged within their limit
    assert 1 <= int(platt[2]) <= 100 and 1 <= it <= 100 and platt[3] == stats[population, ..., 0].sum()
    if T == 0.0:
        assert 0.1 < a < 3.0                                  # a sane slope: greedy labels do depend on logit q0
    want = cal.refit_table(stats, population, min_count, rnd.table.numpy().astype(np.float64))
    assert np.allclose(table, want, rtol=2e-7, atol=0)        # fp32 rounding of the stored table
    assert (np.diff(table, axis=1) >= 0).all() and (table > 0).all() and (table <= 1).all()


def test_refit_fallbacks_and_platt_context():
    # a context in two-scalar mode: rows without data come from the caller's fallback, else from the
    # context's map sampled at the knots
    wl = small("tiny", V=3000, B=4, calib_mode=0)
    rnd = Round(wl, seed=71)
    ts = make_gpu(wl, None, max_batch=rnd.B)
    stats_dev = ts.calib_new_stats()
    table_dev, platt_dev = ts.calib_refit(stats_dev)          # no data at all
    torch.cuda.synchronize()
    knots = np.linspace(LO, HI, cal.KNOTS)
    want = 1 / (1 + np.exp(-(0.67 * knots - 0.46)))
    assert np.allclose(table_dev.cpu().numpy(), np.tile(want, (wl.D, 1)), rtol=3e-7)
    assert platt_dev.cpu().tolist() == [0.0, 0.0, 1.0, 0.0]  # the start: nothing to move for
    fb = torch.rand(wl.D, cal.KNOTS, device="cuda").sort(dim=1).values.clamp_(0.01, 1.0).contiguous()
    table_dev, _ = ts.calib_refit(stats_dev, fallback=fb)
    assert torch.equal(table_dev, fb)
    with pytest.raises(TreeSparkError):
        ts.calib_load_table(fb)                               # not a table-mode context
    with pytest.raises(TreeSparkError):
        ts.calib_refit(stats_dev, population=2)


def test_loaded_table_prices_the_next_round():
    # the loop of Section 3.4 closed on the device: rounds -> statistics -> table -> the next round's trees
    wl = small("serve32", V=12000 + 8, B=8)
    rnd = Round(wl, seed=73)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    stats_dev = ts.calib_new_stats()
    gpu_rounds(ts, rnd, 0.0, seeds=[21, 22, 23, 24, 25, 26], stats_dev=stats_dev)
    table_dev, _ = ts.calib_refit(stats_dev, population=1, min_count=4)
    ts.calib_load_table(table_dev)
    torch.cuda.synchronize()
    new_table = table_dev.cpu()
    assert not torch.equal(new_table, rnd.table)
    orc = make_oracle(wl, new_table)                          # the oracle prices with the same fp32 table
    rnd.theta.fill_(0.05)
    for T in (0.0, 1.0):
        st = check_round(ts, orc, rnd, T, round_seed=33)
        assert st["trees"] == rnd.B
