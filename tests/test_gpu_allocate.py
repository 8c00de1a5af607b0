"""GPU parity of ts_allocate_budget (Section 4, per-request budget allocation) against the CPU oracle:
the same fp32 admission keys go to both sides, so every output is compared bit for bit."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import allocate as alloc
from gpu_harness import ACCEPT_MARGIN, TREE_FLAGS, Round, compare_tree, compare_walk, make_gpu, make_oracle, oracle_trees, to_cpu
from paper_2609_22098_b200 import synth

pytestmark = pytest.mark.gpu

NODE_FIELDS = ("tok", "parent", "depth", "sib_rank", "logS", "q0", "logqT", "logkey", "pop_rank")


def small(name, **kw):
    return dataclasses.replace(synth.WORKLOADS[name], **kw)


def as_oracle_tree(g, b):
    """Request b of a GPU tree (CPU tensors) in the oracle's dict layout, bytes unchanged."""
    t = {"n": int(g["n_nodes"][b])}
    for name in NODE_FIELDS:
        t[name] = g[name][b].numpy().copy()
    t["node_hash"] = g["node_hash"][b].numpy().view(np.uint64).copy()
    t["node_lseT"] = g["node_lseT"][b].numpy().copy()
    t["mask"] = g["mask"][b].numpy().view(np.uint64).copy()
    return t


def assert_cut_equals_oracle(before, after, keep, price_gpu, price):
    B = before["n_nodes"].numel()
    assert after["n_nodes"].tolist() == list(keep)
    if math.isinf(price):
        assert math.isinf(price_gpu) and price_gpu < 0
    else:
        assert price_gpu == np.float32(price)
    for b in range(B):
        want = alloc.trim_tree(as_oracle_tree(before, b), keep[b])
        n = want["n"]
        for name in NODE_FIELDS:
            got = after[name][b, :n].numpy()
            assert np.array_equal(got.view(np.int32), np.asarray(want[name][:n]).view(np.int32)), (b, name)
        assert np.array_equal(after["node_hash"][b, :n + 1].numpy().view(np.uint64), want["node_hash"][:n + 1]), b
        assert np.array_equal(after["node_lseT"][b, :n + 1].numpy().view(np.int32),
                              want["node_lseT"][:n + 1].view(np.int32)), b
        assert np.array_equal(after["mask"][b, :n].numpy().view(np.uint64), want["mask"][:n]), b


def budgets_for(total):
    return sorted({0, 1, total // 3, (2 * total) // 3, max(total - 1, 0), total, total + 10})


@pytest.mark.parametrize("name,kw,T", [
    ("serve32", dict(V=12000 + 8, B=32), 1.0),
    ("serve32", dict(V=12000 + 8, B=32), 0.0),
    ("wide", dict(V=9000, B=8), 0.7),          # Nmax = 256: four mask words, every thread of the cut has a node
    ("decode", dict(V=8000), 1.0),             # one request
    ("sweep", dict(V=6000, B=128), 1.0),       # 128 requests, mixed prices, chain members among them
    ("serve32", dict(V=4000, B=256), 1.0),     # more candidates than the selection keeps in shared memory
])
def test_allocation_and_cut_match_oracle(name, kw, T):
    wl = small(name, **kw)
    rnd = Round(wl, seed=41)
    if name != "sweep":
        rnd.theta.fill_(0.004)                 # large ragged trees
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree0 = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 77)
    torch.cuda.synchronize()
    before = to_cpu(tree0)
    total = int(before["n_nodes"].sum())
    assert total > rnd.B
    price_dev = torch.zeros(4, dtype=torch.float32, device="cuda")
    for budget in budgets_for(total):
        tree = {k: v.clone() for k, v in tree0.items()}
        ts.allocate_budget(tree, budget, price_dev)
        torch.cuda.synchronize()
        keep, price = alloc.water_fill(before["n_nodes"].numpy(), before["logkey"].numpy(), before["pop_rank"].numpy(), budget)
        assert_cut_equals_oracle(before, to_cpu(tree), keep, float(price_dev[0]), price)


@pytest.mark.parametrize("levels", [2, 7])
def test_equal_keys_go_to_the_lowest_request_then_the_earlier_admission(levels):
    # the keys of real trees are replaced by a few distinct values, so that the price falls inside long
    # runs of equal keys spread over many requests
    wl = small("serve32", V=6000, B=48)
    rnd = Round(wl, seed=43)
    rnd.theta.fill_(0.004)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree0 = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 78)
    torch.cuda.synchronize()
    g = to_cpu(tree0)
    rng = np.random.default_rng(levels)
    for b in range(rnd.B):
        n = int(g["n_nodes"][b])
        k = -np.sort(rng.integers(0, levels, size=n)).astype(np.float32) * 0.5   # never increasing in admission order
        for i in range(n):
            g["logkey"][b, i] = float(k[int(g["pop_rank"][b, i])])
    tree0["logkey"].copy_(g["logkey"])
    total = int(g["n_nodes"].sum())
    price_dev = torch.zeros(4, dtype=torch.float32, device="cuda")
    for budget in [1, 5, total // 7, total // 4, total // 2, total - 3]:
        tree = {k: v.clone() for k, v in tree0.items()}
        ts.allocate_budget(tree, budget, price_dev)
        torch.cuda.synchronize()
        keep, price = alloc.water_fill(g["n_nodes"].numpy(), g["logkey"].numpy(), g["pop_rank"].numpy(), budget)
        assert_cut_equals_oracle(g, to_cpu(tree), keep, float(price_dev[0]), price)


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_uniform_price_reproduces_the_theta_rule_on_the_gpu(T):
    # trees grown to the cap and cut to the number of candidates priced >= theta are the trees grown under theta
    wl = small("serve32", V=20000, B=32)
    rnd = Round(wl, seed=47)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    theta = 0.06
    rnd.theta.fill_(theta)
    stopped = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 79))
    rnd.theta.fill_(0.0)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 79)
    full_total = int(tree["n_nodes"].sum())
    budget = int(stopped["n_nodes"].sum())
    assert 0 < budget < full_total
    price_dev = torch.zeros(4, dtype=torch.float32, device="cuda")
    ts.allocate_budget(tree, budget, price_dev)
    torch.cuda.synchronize()
    cut = to_cpu(tree)
    assert float(price_dev[0]) >= math.log(theta) - 1e-6
    assert cut["n_nodes"].tolist() == stopped["n_nodes"].tolist()
    # the two expansions score different parent sets per launch, so their sums are taken in different orders:
    # structure is compared exactly, the floating-point fields under the parity tolerance
    for b in range(rnd.B):
        n = int(cut["n_nodes"][b])
        for name in ("tok", "parent", "depth", "sib_rank", "pop_rank", "mask"):
            assert torch.equal(cut[name][b, :n], stopped[name][b, :n]), (b, name)
        for name in ("logS", "q0", "logqT", "logkey"):
            assert torch.allclose(cut[name][b, :n], stopped[name][b, :n], rtol=1e-5, atol=4e-6), (b, name)
        assert torch.equal(cut["node_hash"][b, :n + 1], stopped["node_hash"][b, :n + 1])


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_verification_of_cut_trees_matches_oracle(T):
    # the cut trees feed ts_verify_tree like any other: the oracle walks its own tree cut to the same sizes
    wl = small("serve32", V=12000 + 8, B=12)
    rnd = Round(wl, seed=53)
    rnd.theta.fill_(0.01)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    orc = make_oracle(wl, rnd.table)
    seed = 80
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, seed)
    torch.cuda.synchronize()
    before = to_cpu(tree)
    budget = int(before["n_nodes"].sum()) // 2
    keep, _ = alloc.water_fill(before["n_nodes"].numpy(), before["logkey"].numpy(), before["pop_rank"].numpy(), budget)
    ts.allocate_budget(tree, budget)
    Z, off = rnd.target_logits(tree)
    verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, seed)
    torch.cuda.synchronize()
    g, v = to_cpu(tree), to_cpu(verdict)
    assert (v["status"] == 0).all()
    c = rnd.cpu()
    otrees, _ = oracle_trees(orc, c["U"], c["A"], c["W"], c["anchor"], c["theta"], T, seed)
    Zc, offc = Z.cpu(), off.cpu()
    Af, Wf = c["A"].float().numpy(), c["W"].float().numpy()
    walked = 0
    for b in range(rnd.B):
        if otrees[b]["flags"] & TREE_FLAGS:
            continue
        ok, _, msg = compare_tree(before, b, otrees[b], wl.D)
        assert ok, msg
        ot = alloc.trim_tree(otrees[b], keep[b])
        ot["flags"] = 0
        ok, _, msg = compare_tree(g, b, ot, wl.D)
        assert ok, msg
        r0 = int(offc[b])
        ov = orc.verify_tree(c["U"][b].float().numpy(), Af, Wf, Zc[r0:r0 + ot["n"] + 1].float().numpy(),
                             int(c["anchor"][b]), ot, T, seed, b, accept_margin=ACCEPT_MARGIN)
        ok, _, msg = compare_walk(v, b, ov, T)
        assert ok, msg
        walked += 1
    assert walked >= rnd.B - 3


def test_argument_errors_launch_nothing():
    wl = small("tiny", V=500, B=2)
    rnd = Round(wl, seed=3)
    ts = make_gpu(wl, rnd.table, max_batch=2)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 0.0, 1)
    torch.cuda.synchronize()
    snap = {k: v.clone() for k, v in tree.items()}
    from paper_2609_22098_b200.binding import TreeSparkError
    with pytest.raises(TreeSparkError):
        ts.allocate_budget(tree, -1)
    bad = dict(tree); bad["logkey"] = None
    with pytest.raises(TreeSparkError):
        ts.allocate_budget(bad, 3)
    torch.cuda.synchronize()
    for k in tree:
        assert torch.equal(tree[k], snap[k], ) or k == "node_lseT"
