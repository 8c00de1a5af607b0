"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the same seeded bytes."""
import dataclasses
import math

import numpy as np
import pytest
import torch
from scipy.stats import chisquare

import oracle
from gpu_harness import (ATOL, RTOL, Round, check_round, close, make_gpu, make_oracle, to_cpu)
from helpers import np_softmax, path_row, tiny_problem, tiny_z_path
from paper_2609_22098_b200 import synth
from paper_2609_22098_b200.binding import TreeSpark

pytestmark = pytest.mark.gpu


def small(name, **kw):
    return dataclasses.replace(synth.WORKLOADS[name], **kw)


# ---------------------------------------------------------------------------------------------
# ts_score_parents
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,r,K", [(1000, 7, 4), (1003, 16, 8), (4096 + 40, 64, 8), (70000, 32, 16), (8, 4, 4), (5, 3, 8),
                                   (9000 + 16, 256, 8), (3000, 200, 4),     # the paper's rank, and one that pads to it
                                   (45000 + 8, 256, 8)])                   # more vocabulary tiles than SMs: a CTA takes several in turn
@pytest.mark.parametrize("T", [0.0, 0.7, 1.0])
@pytest.mark.parametrize("P", [11, 3])   # 3: the few-parents kernel where the context has one
def test_score_parents_matches_oracle(dtype, V, r, K, T, P, test_mode=0):
    if dtype == "f32" and V > 40000 and r == 256:
        pytest.skip("the fp32 kernel keeps r x 128 head values and its W tile in shared memory: at this rank it tiles "
                    "vocabularies up to 32,768 tokens and ts_create answers TS_ERR_UNSUPPORTED beyond")
    wl = small("tiny", V=V, r=r, K=K, D=3, Nmax=16, dtype=dtype, B=3, calib_mode=0)
    rnd = Round(wl, seed=11 + V)
    ts = make_gpu(wl, None, max_batch=3, test_mode=test_mode)
    orc = make_oracle(wl, None)
    g = torch.Generator().manual_seed(V)
    req = torch.randint(0, 3, (P,), generator=g, dtype=torch.int32)
    dep = torch.randint(0, 3, (P,), generator=g, dtype=torch.int32)
    tok = torch.randint(0, V, (P,), generator=g, dtype=torch.int32)
    hsh = torch.randint(0, 2 ** 62, (P,), generator=g, dtype=torch.int64)
    out = to_cpu(ts.score_parents(rnd.U, rnd.A, rnd.W, req.cuda(), dep.cuda(), tok.cuda(), hsh.cuda(), T, seed=99))
    torch.cuda.synchronize()
    c = rnd.cpu()
    Keff = min(K, V)
    checked = 0
    for i in range(P):
        o = orc.score_parent(c["U"][req[i], dep[i]], c["A"][tok[i]], c["W"], T, 99, int(req[i]), int(hsh[i]))
        assert close(out["lse0"][i], o["lse0"]), (i, float(out["lse0"][i]), o["lse0"])
        assert close(out["lseT"][i], o["lseT"]), (i, float(out["lseT"][i]), o["lseT"])
        if o["margins"][0] >= oracle.TOPK_MARGIN:
            assert out["top_tok"][i, :Keff].tolist() == o["top_tok"][:Keff].tolist()
            assert all(close(out["top_logit"][i, j], o["top_logit"][j]) for j in range(Keff))
            checked += 1
        if o["margins"][1] >= oracle.TOPK_MARGIN:
            assert out["draw_tok"][i, :Keff].tolist() == o["draw_tok"][:Keff].tolist(), (i, out["draw_tok"][i], o["draw_tok"])
            assert all(close(out["draw_logit"][i, j], o["draw_logit"][j]) for j in range(Keff))
        if K > V:
            assert (out["top_tok"][i, V:] == -1).all() and (out["draw_tok"][i, V:] == -1).all()
    assert checked >= P - 2


def test_score_parents_more_tiles_than_sms_without_a_tensor_map():
    """Rank 256 on a vocabulary that needs more resident W tiles than there are SMs: with a tensor map the kernel
    streams W through a ring (the case in the list above); without one it keeps the tiled form, a CTA taking its
    tiles in turn and staging W with plain loads."""
    from paper_2609_22098_b200 import binding
    test_score_parents_matches_oracle("bf16", 45000 + 8, 256, 8, 1.0, 11, test_mode=binding.TEST_NO_TMA)


# ---------------------------------------------------------------------------------------------
# full rounds on scaled-down workloads (several tiles, ragged tails, ragged trees)
# ---------------------------------------------------------------------------------------------
CASES = [
    # name, overrides, temperatures, thetas
    ("tiny", dict(), (0.0, 1.0), (0.05,)),
    ("tiny", dict(V=3001, Nmax=40, K=3, D=5), (0.0, 0.8), (0.0, 0.02)),
    ("decode", dict(V=9000 + 24, r=64, B=3), (0.0, 0.7, 1.0), (0.3, 0.1, 0.03)),
    ("serve32", dict(V=20000, B=9), (1.0,), (0.1, 0.0, 1.0)),
    ("wide", dict(V=6000 + 8, B=2, Nmax=256, K=16, D=16, r=128), (0.7, 1.3), (0.01,)),
    ("wide", dict(V=700, B=2, Nmax=70, K=5, D=3, r=9, dtype="f32"), (1.3,), (0.0,)),
]


@pytest.mark.parametrize("name,over,temps,thetas", CASES)
def test_round_matches_oracle(name, over, temps, thetas):
    wl = small(name, **over)
    rnd = Round(wl, seed=1234)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    orc = make_oracle(wl, rnd.table)
    tot = dict(trees=0, trees_exempt=0, walks=0, walks_exempt=0, nodes=0)
    for T in temps:
        for th in thetas:
            rnd.theta.fill_(th)
            for rs in range(3):
                st = check_round(ts, orc, rnd, T, round_seed=1000 + rs)
                for k in tot:
                    tot[k] += st[k]
    # measured over the whole suite: 0.9 % of trees and 0.5 % of walks are exempt (none by the accept margin); a
    # test of a few dozen rounds may see a handful
    assert tot["trees_exempt"] <= 0.03 * tot["trees"] + 3
    assert tot["walks_exempt"] <= 0.03 * tot["walks"] + 3
    assert tot["nodes"] > 0


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_empty_trees_only_draw_the_bonus_token(T):
    """A price no edge can meet (but below the chain sentinel): every tree is empty, verification commits
    nothing and emits the bonus token from the root row alone."""
    wl = small("serve32", V=9000 + 8, B=7)
    rnd = Round(wl, seed=77)
    rnd.theta.fill_(0.99999)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    orc = make_oracle(wl, rnd.table)
    for rs in range(3):
        st = check_round(ts, orc, rnd, T, round_seed=300 + rs)
        assert st["trees"] == rnd.B and st["nodes"] == 0 and st["acc"] == 0


def test_tiny_reference_config_100_rounds():
    """The tiny all-fp32 reference configuration at full size: 100 rounds at T = 0 and T = 1."""
    wl = synth.WORKLOADS["tiny"]
    rnd = Round(wl, seed=7)
    ts = make_gpu(wl, rnd.table, max_batch=1)
    orc = make_oracle(wl, rnd.table)
    for T in wl.temps:
        tot = dict(trees=0, trees_exempt=0, walks=0, walks_exempt=0, nodes=0)
        for rs in range(100):
            st = check_round(ts, orc, rnd, T, round_seed=5000 + rs, want_edge=(rs % 10 == 0))
            for k in tot:
                tot[k] += st[k]
        assert tot["trees_exempt"] <= 4 and tot["walks_exempt"] <= 4, tot
        assert tot["nodes"] >= 100


def test_back_to_back_rounds_reproduce_bitwise():
    """Rounds queued back to back on one stream, no host synchronisation in between, alternating between two
    input sets: the kernels of a round start while the previous kernel is still finishing (chained launches),
    so every result is compared bit for bit with the one the same inputs gave when run alone."""
    wl = small("serve32", V=20000 + 8, B=6)
    sets = [Round(wl, seed=300), Round(wl, seed=301)]
    ts = make_gpu(wl, sets[0].table, max_batch=6)
    alone = []
    for rnd in sets:
        tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 42)
        Z, off = rnd.target_logits(tree)
        verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, 1.0, 42)
        torch.cuda.synchronize()
        alone.append((Z, off, {k: v.clone() for k, v in to_cpu(tree).items()}, {k: v.clone() for k, v in to_cpu(verdict).items()}))
    queued = []
    for i in range(300):
        rnd = sets[i % 2]
        Z, off, _, _ = alone[i % 2]
        tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 42)
        verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, 1.0, 42)
        queued.append((tree, verdict))   # every call has its own output buffers
    torch.cuda.synchronize()
    for i, (tree, verdict) in enumerate(queued):
        _, _, t0, v0 = alone[i % 2]
        n = t0["n_nodes"]
        assert torch.equal(tree["n_nodes"].cpu(), n)
        for b in range(len(n)):
            nb = int(n[b])
            for key in ("tok", "parent", "depth", "sib_rank", "logS", "q0", "logqT"):
                assert torch.equal(tree[key].cpu()[b, :nb], t0[key][b, :nb]), (i, b, key)
            assert torch.equal(tree["mask"].cpu()[b, :nb], t0["mask"][b, :nb]), (i, b)
        for key in ("acc_len", "bonus_tok", "status"):
            assert torch.equal(verdict[key].cpu(), v0[key]), (i, key)
        for b in range(len(n)):
            L = int(v0["acc_len"][b])
            assert torch.equal(verdict["acc_tok"].cpu()[b, :L], v0["acc_tok"][b, :L]), (i, b)


@pytest.mark.parametrize("dtype,mode", [("f32", 0), ("bf16", "TEST_FORCE_FMA"), ("bf16", 0)])
def test_a_request_that_accepts_a_full_depth_path_beside_requests_that_reject(dtype, mode):
    """The last request of the batch drafts a chain of depth D (theta = 1) against a target equal to its drafter,
    so its walk accepts all D tokens and draws its bonus token at a leaf of depth D, which has no base-logit row
    (rows are depths 0 .. D-1); its neighbours in the same reduction groups reject early and ask for proposal
    residuals.  The reductions of the walk (the fused-multiply-add path for fp32 inputs, and for bf16 inputs under
    the switch that forces it; the tensor-core path otherwise) must not touch a base-logit row for the leaf."""
    from paper_2609_22098_b200 import binding
    wl = small("serve32", V=12000 + 8, B=5, D=4, dtype=dtype)
    rnd = Round(wl, seed=321)
    rnd.theta[rnd.B - 1] = 1.0
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B, test_mode=getattr(binding, mode) if mode else 0)
    orc = make_oracle(wl, rnd.table)
    full = 0
    for seed in (3, 4, 5):
        st = check_round(ts, orc, rnd, 1.0, seed, sigma_by_req={rnd.B - 1: 0.0})
        assert st["n_nodes"].get(rnd.B - 1, wl.D) == wl.D
        full += 1 if st["acc_len"].get(rnd.B - 1) == wl.D else 0
    assert full >= 1, "no round accepted the whole chain: the case under test was not reached"


@pytest.mark.parametrize("mode", ["TEST_FORCE_FMA", "TEST_NO_TMA", "TEST_NO_FEW", "TEST_NO_SEED", "TEST_PERSIST", "TEST_NO_UMMA", "TEST_NO_TAIL"])
def test_alternative_kernel_paths_match_oracle(mode):
    """bf16 inputs on the fp32-FMA kernels; the tensor-core kernels with W staged by plain loads (the path
    taken when no tensor map can be encoded); every level on the tile kernel; the tile kernel without seeded
    bounds; every level inside one cooperative launch, or none of them (by default the levels from the fifth on): chosen by the library's
    test switches."""
    from paper_2609_22098_b200 import binding
    wl = small("serve32", V=20000, B=5)
    rnd = Round(wl, seed=77)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B, test_mode=getattr(binding, mode))
    orc = make_oracle(wl, rnd.table)
    for T in (0.0, 1.0):
        st = check_round(ts, orc, rnd, T, round_seed=900)
        assert st["nodes"] > 0


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_round_replayed_from_a_cuda_graph_equals_direct_calls(T):
    """The hot calls allocate nothing and never synchronise: a whole round (every launch of expand and
    verify, cooperative walk included) is captured in a CUDA graph and its replays give the direct results,
    also after the inputs behind the captured pointers have changed."""
    wl = small("serve32", V=20000, B=6)
    rnd = Round(wl, seed=66)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree, verdict = ts.alloc_tree(rnd.B), ts.alloc_verdict(rnd.B)
    U = rnd.U.clone()
    ts.expand_tree(U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 21, out=tree)   # also encodes the tensor map before capture
    Z, off = rnd.target_logits(tree)
    ts.verify_tree(U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, 21, out=verdict)
    torch.cuda.synchronize()
    want = (to_cpu(tree), to_cpu(verdict))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ts.expand_tree(U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 21, out=tree)
        ts.verify_tree(U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, 21, out=verdict)
    torch.cuda.current_stream().wait_stream(side)

    def same(a, b):
        n = a["n_nodes"]
        ok = torch.equal(a["n_nodes"], b["n_nodes"])
        for bb in range(rnd.B):
            for k in ("tok", "parent", "depth", "logS", "pop_rank"):
                ok = ok and torch.equal(a[k][bb, :int(n[bb])], b[k][bb, :int(n[bb])])
        return ok

    for _ in range(3):
        for t in list(tree.values()) + list(verdict.values()):
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        got = (to_cpu(tree), to_cpu(verdict))
        assert same(want[0], got[0])
        for k in ("acc_len", "acc_tok", "bonus_tok", "status"):
            assert torch.equal(want[1][k], got[1][k]), k
    # other base logits behind the same pointer: the replay follows them (trees change), as a direct call does
    U.copy_(Round(wl, seed=67).U)
    g.replay()
    torch.cuda.synchronize()
    replayed = to_cpu(tree)
    direct = to_cpu(ts.expand_tree(U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 21))
    assert same(direct, replayed) and not torch.equal(replayed["tok"], want[0]["tok"])


def test_host_round_two_in_flight_equals_one_at_a_time():
    """The host-buffer round: submit / collect with two rounds in flight returns what run() returns."""
    from paper_2609_22098_b200.binding import HostRound
    wl = small("serve32", V=20000 + 16, B=5)
    rnds = [Round(wl, seed=500 + i) for i in range(3)]
    ts = make_gpu(wl, rnds[0].table, max_batch=5)
    A, W = rnds[0].A, rnds[0].W   # one head for all three input sets
    host = []
    for rnd in rnds:
        tree = ts.expand_tree(rnd.U, A, W, rnd.anchor, rnd.theta, 1.0, 9)   # the tree the round below will build
        Z, off = rnd.target_logits(tree)                                      # one target row per node of that tree
        host.append(HostRound.pin_inputs(rnd.U, rnd.anchor, rnd.theta, Z, off))
    hr = HostRound(ts, 5, max(int(h["Z"].shape[0]) for h in host))
    ref = []
    for h in host:
        out = hr.run(h, A, W, 1.0, 9)
        ref.append({k: v.clone() for k, v in out.items()})
    got = []
    for i in range(9):
        hr.submit(host[i % 3], A, W, 1.0, 9)
        if i > 0:
            got.append({k: v.clone() for k, v in hr.collect().items()})
    got.append({k: v.clone() for k, v in hr.collect().items()})
    for i, g in enumerate(got):
        r = ref[i % 3]
        n = r["n_nodes"]
        assert torch.equal(g["n_nodes"], n) and torch.equal(g["acc_len"], r["acc_len"]) and torch.equal(g["bonus_tok"], r["bonus_tok"])
        for b in range(5):
            assert torch.equal(g["tok"][b, :int(n[b])], r["tok"][b, :int(n[b])])
            assert torch.equal(g["acc_tok"][b, :int(r["acc_len"][b])], r["acc_tok"][b, :int(r["acc_len"][b])])


@pytest.mark.parametrize("which", ["marginal_tree", "raw_priority"])
def test_ablation_settings_match_oracle(which):
    """Two of the paper's ablation axes need no code of their own: the marginal tree (scores from the base
    logits only) is a zero head matrix A, and the uncalibrated sum-of-log-q priority is the Platt map with
    a = 1, b = 0 (p-hat = q_0).  Both must match the oracle like any other setting."""
    wl = small("serve32", V=12000 + 8, B=4, calib_mode=0)
    rnd = Round(wl, seed=910)
    a, b = (0.67, -0.46)
    if which == "marginal_tree":
        rnd.A.zero_()
    else:
        a, b = 1.0, 0.0
    ts = TreeSpark(wl.V, wl.D, wl.r, wl.K, wl.Nmax, rnd.B, dtype=wl.torch_dtype, calib_mode=0, platt_a=a, platt_b=b)
    orc = oracle.Oracle(wl.V, wl.D, wl.r, wl.K, wl.Nmax, calib_mode=0, platt_a=a, platt_b=b)
    rnd.theta.fill_(0.02)
    for T in (0.0, 1.0):
        st = check_round(ts, orc, rnd, T, round_seed=31)
        assert st["trees"] == rnd.B


@pytest.mark.parametrize("calib_mode", [0, 1])
def test_tempered_calibrator_switch_matches_oracle(calib_mode):
    """The ablation that feeds the calibrator q_T instead of q0 (Section 5.5), against the oracle's switch;
    the trees must also differ from the method's at T != 1 (the switch does something) and not at T = 0."""
    wl = small("serve32", V=12000 + 8, B=6, calib_mode=calib_mode)
    rnd = Round(wl, seed=920)
    table = rnd.table if calib_mode == 1 else None
    ts = make_gpu(wl, table, max_batch=rnd.B)
    plain = {T: to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 37)) for T in (0.0, 0.6)}
    ts.set_ablation(1)
    orc = oracle.Oracle(wl.V, wl.D, wl.r, wl.K, wl.Nmax, calib_mode=calib_mode, calib_input=1,
                        calib_table=None if table is None else table.numpy().astype(np.float64))
    for T in (0.0, 0.6, 1.0):
        st = check_round(ts, orc, rnd, T, round_seed=37)
        assert st["trees"] == rnd.B
    fed = {T: to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 37)) for T in (0.0, 0.6)}
    assert torch.equal(fed[0.0]["logS"], plain[0.0]["logS"]) and torch.equal(fed[0.0]["n_nodes"], plain[0.0]["n_nodes"])
    assert int(fed[0.6]["n_nodes"].sum()) > int(plain[0.6]["n_nodes"].sum())   # sharper proposal, larger trees
    ts.set_ablation(0)
    back = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 0.6, 37))
    assert torch.equal(back["n_nodes"], plain[0.6]["n_nodes"])
    with pytest.raises(Exception):
        ts.set_ablation(2)


@pytest.mark.parametrize("dtype,V,B", [("bf16", 20000 + 8, 6), ("f32", 20000 + 8, 6),
                                       ("bf16", 60000 + 8, 4)])   # a range of W that no longer fits shared memory: the walk streams it
def test_round_at_the_papers_own_shape_matches_oracle(dtype, V, B):
    # rank 256, block of 7, 56 nodes, 8 siblings (Section 5.1), on a vocabulary the oracle finishes quickly
    wl = small("serve32", V=V, r=256, D=7, Nmax=56, K=8, B=B, dtype=dtype)
    rnd = Round(wl, seed=97)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    orc = make_oracle(wl, rnd.table)
    rnd.theta.fill_(0.03)
    for T in (0.0, 1.0):
        st = check_round(ts, orc, rnd, T, round_seed=41)
        assert st["trees"] == rnd.B and st["nodes"] > 4 * rnd.B


def test_chain_sentinel_and_mixed_prices():
    wl = small("serve32", V=5000, B=6)
    rnd = Round(wl, seed=21)
    rnd.theta.copy_(torch.tensor([1.0, 0.1, 2.0, 0.0, 0.5, 1.0]))
    ts = make_gpu(wl, rnd.table, max_batch=6)
    orc = make_oracle(wl, rnd.table)
    check_round(ts, orc, rnd, 1.0, 77)
    tree = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 0.0, 78))
    for b in (0, 2, 5):
        assert int(tree["n_nodes"][b]) == wl.D
        assert tree["depth"][b, :wl.D].tolist() == list(range(1, wl.D + 1))
        assert tree["parent"][b, :wl.D].tolist() == list(range(-1, wl.D - 1))
    assert int(tree["n_nodes"][3]) == wl.Nmax


def test_argument_validation_returns_errors_without_launching():
    from paper_2609_22098_b200.binding import TreeSparkError
    wl = small("tiny", V=512)
    rnd = Round(wl, seed=3)
    ts = make_gpu(wl, rnd.table, max_batch=1)
    with pytest.raises(TreeSparkError):
        ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, -1.0, 1)
    with pytest.raises(TreeSparkError):
        ts.expand_tree(rnd.U.view(-1)[1:], rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 1)   # misaligned
    with pytest.raises(TreeSparkError):
        TreeSpark(512, 4, 16, 32, 16, 1)                                                   # K > 16
    small_ws = ts.ws_bytes
    ts.ws_bytes = 1024
    with pytest.raises(TreeSparkError):
        ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 1)
    ts.ws_bytes = small_ws
    bad = rnd.anchor.clone(); bad[0] = wl.V + 5
    tree = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, bad, rnd.theta, 1.0, 1))
    assert int(tree["status"][0]) == -1 and int(tree["n_nodes"][0]) == 0


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_non_finite_base_logits_are_reported_for_their_request_only(dtype):
    """A NaN row or an infinite logit cannot be scored: the request's status says so, the call returns, and
    the other requests of the batch get exactly the trees they get without the bad neighbour."""
    wl = small("serve32", V=12000 + 8, B=5, dtype=dtype)
    rnd = Round(wl, seed=930)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    clean = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 5))
    U = rnd.U.clone()
    U[1, 0, :] = float("nan")                                 # a whole row
    U[3, 0, 777] = float("inf")                               # one token
    bad = to_cpu(ts.expand_tree(U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 5))
    torch.cuda.synchronize()
    assert bad["status"].tolist() == [0, -7, 0, -7, 0]
    for b in (0, 2, 4):
        n = int(clean["n_nodes"][b])
        assert int(bad["n_nodes"][b]) == n
        for name in ("tok", "parent", "depth", "sib_rank", "pop_rank"):
            assert torch.equal(bad[name][b, :n], clean[name][b, :n]), (b, name)
        # (the two calls score different parent sets per launch: sums in another order, last-place differences)
        assert torch.allclose(bad["logS"][b, :n], clean["logS"][b, :n], rtol=1e-5, atol=4e-6)
    again = to_cpu(ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 5))   # the context is unharmed
    assert torch.equal(again["n_nodes"], clean["n_nodes"]) and torch.equal(again["tok"], clean["tok"])
    assert (again["status"] == 0).all()


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_non_finite_target_logits_are_reported_for_their_request_only(T):
    """A NaN anywhere in a target row of a request: that request is not walked (status, no accepted
    tokens, no bonus token), the others get exactly the verdict they get without it."""
    wl = small("serve32", V=12000 + 8, B=5)
    rnd = Round(wl, seed=940)
    rnd.theta.fill_(0.03)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 6)
    Z, off = rnd.target_logits(tree)
    clean = to_cpu(ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, 6))
    assert (clean["status"] == 0).all()
    offc = off.cpu()
    Zb = Z.clone()
    Zb[int(offc[1]), 4321] = float("nan")                     # the root row of request 1
    Zb[int(offc[4]) - 1, 17] = float("nan")                   # the last row of request 3
    bad = to_cpu(ts.verify_tree(rnd.U, rnd.A, rnd.W, Zb, off, rnd.anchor, tree, T, 6))
    torch.cuda.synchronize()
    assert bad["status"].tolist() == [0, -7, 0, -7, 0]
    for b in (1, 3):
        assert int(bad["acc_len"][b]) == 0 and int(bad["bonus_tok"][b]) == -1
        assert (bad["edge_stat"][b, :int(tree["n_nodes"][b])] == 0).all()
    for b in (0, 2, 4):
        for name in ("acc_len", "acc_node", "acc_tok", "bonus_tok", "flags"):
            assert torch.equal(bad[name][b], clean[name][b]), (b, name)
        n = int(tree["n_nodes"][b])
        assert torch.equal(bad["edge_stat"][b, :n], clean["edge_stat"][b, :n])
    again = to_cpu(ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, 6))   # the context is unharmed
    for name in ("status", "acc_len", "acc_tok", "bonus_tok"):
        assert torch.equal(again[name], clean[name]), name


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_impossible_node_count_is_refused_for_its_request_only(T):
    wl = small("serve32", V=12000 + 8, B=4)
    rnd = Round(wl, seed=950)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 8)
    Z, off = rnd.target_logits(tree)
    clean = to_cpu(ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, 8))
    broken = dict(tree)
    broken["n_nodes"] = tree["n_nodes"].clone()
    broken["n_nodes"][2] = wl.Nmax + 7
    broken["n_nodes"][0] = -3
    got = to_cpu(ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, broken, T, 8))
    torch.cuda.synchronize()
    assert got["status"].tolist() == [-1, 0, -1, 0]
    assert got["acc_len"][[0, 2]].tolist() == [0, 0] and got["bonus_tok"][[0, 2]].tolist() == [-1, -1]
    for b in (1, 3):
        for name in ("acc_len", "acc_tok", "bonus_tok"):
            assert torch.equal(got[name][b], clean[name][b]), (b, name)


# ---------------------------------------------------------------------------------------------
# losslessness on the GPU path itself (Proposition 1), tiny vocabulary, many requests per call
# ---------------------------------------------------------------------------------------------
def test_gpu_losslessness_chi_square():
    V, D, r, K, N, T, theta = 8, 3, 4, 4, 12, 1.0, 0.05
    U, A, W = tiny_problem(60, V, D, r, u_std=1.5)
    Zp = tiny_z_path(61, U, A, W, D, sigma=1.0, anchor=3)
    B = 4096
    ts = TreeSpark(V, D, r, K, N, B, dtype=torch.float32)
    Ud = torch.from_numpy(U[:D]).cuda().unsqueeze(0).expand(B, D, V).contiguous()
    Ad, Wd = torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda()
    Zpd = torch.from_numpy(Zp).cuda()
    anchor = torch.full((B,), 3, dtype=torch.int32, device="cuda")
    th = torch.full((B,), theta, dtype=torch.float32, device="cuda")
    off_len = torch.tensor([sum(V ** k for k in range(d)) for d in range(D + 1)], device="cuda")
    h1 = torch.zeros(V, dtype=torch.int64, device="cuda")
    h2 = torch.zeros(V, V, dtype=torch.int64, device="cuda")
    calls = 64
    for c in range(calls):
        tree = ts.expand_tree(Ud, Ad, Wd, anchor, th, T, seed=900 + c)
        n = tree["n_nodes"].long()
        # path index of every node: fold tokens along parent pointers (depth <= 3)
        tok, par, dep = tree["tok"].long(), tree["parent"].long(), tree["depth"].long()
        idx = tok.clone()
        mult = torch.full_like(idx, V)
        cur = par.clone()
        for _ in range(D - 1):
            has = cur >= 0
            ptok = torch.gather(tok, 1, cur.clamp(min=0))
            idx = torch.where(has, idx + ptok * mult, idx)
            mult = torch.where(has, mult * V, mult)
            cur = torch.where(has, torch.gather(par, 1, cur.clamp(min=0)), cur)
        prow = off_len[dep.clamp(0, D)] + idx
        rows = []
        offs = torch.zeros(B + 1, dtype=torch.int64, device="cuda")
        offs[1:] = torch.cumsum(n + 1, 0)
        total = int(offs[-1])
        Z = torch.empty(total, V, device="cuda")
        Z[offs[:-1]] = Zpd[0]
        ar = torch.arange(N, device="cuda").unsqueeze(0).expand(B, N)
        valid = ar < n.unsqueeze(1)
        dst = (offs[:-1].unsqueeze(1) + 1 + ar)[valid]
        Z[dst] = Zpd[prow[valid]]
        v = ts.verify_tree(Ud, Ad, Wd, Z, offs, anchor, tree, T, seed=900 + c, edge_stat=False)
        assert int(v["status"].abs().max()) == 0
        L = v["acc_len"].long()
        first = torch.where(L >= 1, v["acc_tok"][:, 0].long(), v["bonus_tok"].long())
        h1 += torch.bincount(first, minlength=V)
        second = torch.where(L >= 2, v["acc_tok"][:, 1].long(), v["bonus_tok"].long())
        sel = L >= 1
        h2 += torch.bincount(first[sel] * V + second[sel], minlength=V * V).reshape(V, V)
    trials = B * calls
    h1 = h1.cpu().numpy(); h2 = h2.cpu().numpy()
    p_root = np_softmax(Zp[0].astype(np.float64), T)
    assert h1.sum() == trials
    assert chisquare(h1, p_root * trials).pvalue > 1e-3
    checked = 0
    for x1 in range(V):
        nrow = int(h2[x1].sum())
        if nrow < 5000:
            continue
        p2 = np_softmax(Zp[path_row((x1,), V)].astype(np.float64), T)
        assert chisquare(h2[x1], p2 * nrow).pvalue > 1e-4
        checked += 1
    assert checked >= 2


@pytest.mark.parametrize("T", [0.0, 1.0])
@pytest.mark.parametrize("persist", [True, False])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(T, persist):
    """Bounded device-side waits: with the test switch that makes barriers expect one arrival more than will ever
    come (and shortens the limit to a few thousand polls) the kernels give up, every call returns, the requests
    are reported with TS_ERR_TIMEOUT, and the same context then runs an ordinary round correctly."""
    from paper_2609_22098_b200 import binding
    wl = small("serve32", V=20000, B=6)
    rnd = Round(wl, seed=91)
    base = binding.TEST_PERSIST if persist else 0
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B, test_mode=base)
    orc = make_oracle(wl, rnd.table)
    good = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 5)
    Z, off = rnd.target_logits(good)
    torch.cuda.synchronize()
    ts.set_test_mode(base | binding.TEST_SHORT_WAITS | binding.TEST_LOST_ARRIVAL)
    bad_tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, 5)
    torch.cuda.synchronize()
    assert (bad_tree["status"].cpu() == -5).all(), bad_tree["status"]          # TS_ERR_TIMEOUT, and the call came back
    if T > 0:
        bad_verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, good, T, 5)
        torch.cuda.synchronize()
        assert (bad_verdict["status"].cpu() == -5).all(), bad_verdict["status"]
    ts.set_test_mode(base)
    for rs in range(2):
        st = check_round(ts, orc, rnd, T, round_seed=40 + rs)
        assert st["nodes"] > 0
