"""Test-side harness: run one round on the CUDA path and on the CPU oracle with the same bytes and
compare under the stated tolerances.  Imported by the GPU tests, the smoke check and the bench's
parity check; nothing in the product imports it."""
from __future__ import annotations

import atexit
import json
import os

import numpy as np
import torch

import oracle
from paper_2609_22098_b200 import synth
from paper_2609_22098_b200.binding import TreeSpark

# Tolerances: probabilities and log-survivals are accumulated in fp32 on
# the GPU and compared at 1e-5 relative plus an absolute floor of two fp32 ulps of a logit of
# magnitude <= 32 (the inputs of every scalar are such logits).
RTOL = 1e-5
ATOL = 4e-6
ACCEPT_MARGIN = 1e-6   # |u - rho| below this exempts an accept test (the stated allowance; no walk of the suite sits in [1e-6, 1e-5))
TREE_FLAGS = oracle.FLAG_NEAR_TOPK | oracle.FLAG_NEAR_THETA | oracle.FLAG_NEAR_CAP
WALK_FLAGS = oracle.FLAG_NEAR_ACCEPT | oracle.FLAG_NEAR_CDF | oracle.FLAG_ZERO_MASS


# Every compared round adds to these counts; when TS_PARITY_REPORT_DIR names a folder they are written there at
# exit, so that the exemption rates behind the tolerances can be read off a test run (tests still assert ceilings).
PARITY_TOTALS = dict(trees=0, trees_exempt=0, walks=0, walks_exempt=0, accept_band_walks=0, accept_band_disagree=0)
_BY_FLAG = {}


def _dump_totals():
    out = os.environ.get("TS_PARITY_REPORT_DIR", "")
    if PARITY_TOTALS["trees"] and out and os.path.isdir(out):
        with open(os.path.join(out, f"parity_exemptions_{os.getpid()}.json"), "w") as f:
            json.dump(dict(totals=PARITY_TOTALS, by_flag=_BY_FLAG), f)


atexit.register(_dump_totals)


def _count_flags(flags, which):
    for name in ("NEAR_TOPK", "NEAR_THETA", "NEAR_CAP", "NEAR_ACCEPT", "NEAR_CDF", "ZERO_MASS"):
        if flags & getattr(oracle, "FLAG_" + name) & which:
            _BY_FLAG[name] = _BY_FLAG.get(name, 0) + 1


def make_oracle(wl, table):
    return oracle.Oracle(wl.V, wl.D, wl.r, wl.K, wl.Nmax, calib_mode=wl.calib_mode,
                         calib_table=None if table is None else table.numpy().astype(np.float64))


def make_gpu(wl, table, max_batch, test_mode=0):
    return TreeSpark(wl.V, wl.D, wl.r, wl.K, wl.Nmax, max_batch, dtype=wl.torch_dtype, calib_mode=wl.calib_mode,
                     calib_table=table, test_mode=test_mode)


def close(a, b, rtol=RTOL, atol=ATOL):
    return abs(float(a) - float(b)) <= atol + rtol * max(abs(float(a)), abs(float(b)))


def oracle_trees(orc, U, A, W, anchor, theta, T, seed, reqs=None, threads=None):
    """Oracle expansion for the listed requests (default all).  U is [B][>=D][V] on the CPU."""
    Af, Wf = A.float().numpy(), W.float().numpy()
    reqs = list(range(U.shape[0])) if reqs is None else list(reqs)
    def one(b):
        return orc.expand_tree(U[b].float().numpy(), Af, Wf, int(anchor[b]), float(theta[b]), T, seed, b)
    out, used = oracle.run_batch(one, reqs, threads)
    return dict(zip(reqs, out)), used


def compare_tree(g, b, o, D):
    """GPU tree (dict of CPU tensors) vs oracle tree for request b.  Returns (ok, exempt, message)."""
    if o["flags"] & TREE_FLAGS:
        return True, True, "flagged"
    n = int(o["n"])
    if int(g["n_nodes"][b]) != n:
        return False, False, f"req {b}: n_nodes {int(g['n_nodes'][b])} != {n}"
    for name, key in (("tok", "tok"), ("parent", "parent"), ("depth", "depth"), ("sib_rank", "sib_rank")):
        if not np.array_equal(g[name][b, :n].numpy(), o[key][:n]):
            return False, False, f"req {b}: {name} differs: {g[name][b, :n].tolist()} vs {o[key][:n].tolist()}"
    if not np.array_equal(g["mask"][b, :n].numpy().view(np.uint64), o["mask"][:n]):
        return False, False, f"req {b}: mask differs"
    if not np.array_equal(g["node_hash"][b, :n + 1].numpy().view(np.uint64), o["node_hash"][:n + 1]):
        return False, False, f"req {b}: node_hash differs"
    if not np.array_equal(g["pop_rank"][b, :n].numpy(), o["pop_rank"][:n]):
        return False, False, f"req {b}: pop_rank differs"
    for i in range(n):
        for name in ("logS", "q0", "logqT", "logkey"):
            if not close(g[name][b, i], o[name][i]):
                return False, False, f"req {b} node {i}: {name} {float(g[name][b, i])!r} vs {o[name][i]!r}"
    # what the header promises about the two outputs whose coverage differs from the oracle's (the oracle scores
    # every admitted node above depth D; the library only the nodes that reach a level's parent list)
    has_child = np.zeros(n + 1, dtype=bool)          # slot 0 = root
    has_child[np.asarray(o["parent"][:n], dtype=np.int64) + 1] = True
    if n > 0 and "n_scored" in g and int(g["n_scored"][b]) < int(has_child.sum()):
        return False, False, f"req {b}: n_scored {int(g['n_scored'][b])} < nodes with children {int(has_child.sum())}"
    if "node_lseT" in g:
        lse = g["node_lseT"][b, :n + 1].numpy()
        if not np.isfinite(lse[has_child]).all():
            return False, False, f"req {b}: node_lseT not finite at a node with children"
        if "node_lseT" in o:
            ol = np.asarray(o["node_lseT"][:n + 1], dtype=np.float64)
            for i in np.nonzero(has_child)[0]:
                if not close(lse[i], ol[i]):
                    return False, False, f"req {b} slot {i}: node_lseT {float(lse[i])!r} vs {float(ol[i])!r}"
    return True, False, ""


def compare_walk(v, b, ov, T):
    """GPU verdict (dict of CPU tensors) vs oracle verdict."""
    if ov["flags"] & WALK_FLAGS:
        return True, True, "flagged"
    L = int(ov["acc_len"])
    if int(v["acc_len"][b]) != L:
        return False, False, f"req {b}: acc_len {int(v['acc_len'][b])} != {L}"
    if v["acc_tok"][b, :L].tolist() != ov["acc_tok"][:L].tolist() or v["acc_node"][b, :L].tolist() != ov["acc_node"][:L].tolist():
        return False, False, f"req {b}: accepted path differs"
    if int(v["bonus_tok"][b]) != int(ov["bonus"]):
        return False, False, f"req {b}: bonus {int(v['bonus_tok'][b])} != {int(ov['bonus'])}"
    return True, False, ""


def to_cpu(d):
    return {k: t.detach().cpu() for k, t in d.items()}


class Round:
    """Inputs of one workload instance, resident on the GPU, with CPU copies for the oracle."""

    def __init__(self, wl, seed, B=None, theta=None, table_kind="fit", device="cuda", gen_device=None):
        self.wl = wl
        self.B = wl.B if B is None else B
        gen_device = gen_device or device
        self.gen_device, self.device = gen_device, device
        self.table = synth.make_calibration_table(wl, seed + 4, table_kind) if wl.calib_mode == 1 else None
        A, W = synth.make_head(wl, seed + 1, gen_device)
        Ufull = synth.make_base_logits(wl, seed + 2, gen_device, B=self.B)
        self.A, self.W, self.Ufull = A.to(device), W.to(device), Ufull.to(device)
        self.U = self.Ufull[:, :wl.D].contiguous()
        self.anchor = synth.make_anchor(wl, seed + 3, B=self.B).to(device)
        self.theta = synth.make_theta(wl, B=self.B, theta=theta).to(device)
        self.seed = seed

    def cpu(self):
        return dict(A=self.A.cpu(), W=self.W.cpu(), U=self.Ufull.cpu(), anchor=self.anchor.cpu(), theta=self.theta.cpu())

    def target_logits(self, tree, sigma=None):
        """Z for the given (GPU) tree; generated once, on the device the inputs were generated on."""
        wl = self.wl
        if str(self.gen_device) == "cpu" and str(self.device) != "cpu":
            c = self.cpu()
            Z, off = synth.make_target_logits(wl, self.seed + 5, c["U"], c["A"], c["W"], c["anchor"], tree["n_nodes"].cpu(),
                                              tree["tok"].cpu(), tree["depth"].cpu(), tree["node_hash"].cpu(), sigma=sigma)
            return Z.to(self.device), off.to(self.device)
        return synth.make_target_logits(wl, self.seed + 5, self.Ufull, self.A, self.W, self.anchor, tree["n_nodes"],
                                        tree["tok"], tree["depth"], tree["node_hash"], sigma=sigma)


def check_round(ts, orc, rnd: Round, T, round_seed, reqs=None, want_edge=True, threads=None, sigma_by_req=None):
    """Expand + verify on the GPU, then the oracle on the same bytes for `reqs`; returns statistics.
    Raises AssertionError on any mismatch outside the flagged near-ties.  sigma_by_req = {request: sigma}
    regenerates those requests' target rows with another noise level (0: the target is the drafter)."""
    wl = rnd.wl
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, T, round_seed)
    Z, off = rnd.target_logits(tree)
    for b, sg in (sigma_by_req or {}).items():
        Z2, _ = rnd.target_logits(tree, sigma=sg)
        Z[int(off[b]):int(off[b + 1])] = Z2[int(off[b]):int(off[b + 1])]
        del Z2
    verdict = ts.verify_tree(rnd.U, rnd.A, rnd.W, Z, off, rnd.anchor, tree, T, round_seed)
    torch.cuda.synchronize()
    g, v = to_cpu(tree), to_cpu(verdict)
    assert (g["status"] == 0).all(), g["status"]
    assert (v["status"] == 0).all(), v["status"]
    c = rnd.cpu()
    reqs = list(range(rnd.B)) if reqs is None else list(reqs)
    otrees, used = oracle_trees(orc, c["U"], c["A"], c["W"], c["anchor"], c["theta"], T, round_seed, reqs, threads)
    Zc, offc = Z.cpu(), off.cpu()
    Af, Wf = c["A"].float().numpy(), c["W"].float().numpy()
    stats = dict(trees=0, trees_exempt=0, walks=0, walks_exempt=0, nodes=0, acc=0, threads=used, acc_len={}, n_nodes={})

    def verify_one(b):
        o = otrees[b]
        r0 = int(offc[b])
        return orc.verify_tree(c["U"][b].float().numpy(), Af, Wf, Zc[r0:r0 + o["n"] + 1].float().numpy(),
                               int(c["anchor"][b]), o, T, round_seed, b, accept_margin=ACCEPT_MARGIN,
                               want_edge_stat=want_edge)

    ok_reqs = []
    for b in reqs:
        ok, exempt, msg = compare_tree(g, b, otrees[b], wl.D)
        assert ok, msg
        stats["trees"] += 1
        stats["nodes"] += int(otrees[b]["n"])
        if exempt:
            stats["trees_exempt"] += 1
            _count_flags(otrees[b]["flags"], TREE_FLAGS)
        else:
            ok_reqs.append(b)
    overd, _ = oracle.run_batch(verify_one, ok_reqs, threads)
    for b, ov in zip(ok_reqs, overd):
        ok, exempt, msg = compare_walk(v, b, ov, T)
        assert ok, msg
        stats["walks"] += 1
        stats["acc"] += int(ov["acc_len"])
        stats["acc_len"][b] = int(v["acc_len"][b])
        stats["n_nodes"][b] = int(g["n_nodes"][b])
        if exempt:
            stats["walks_exempt"] += 1
            _count_flags(ov["flags"], WALK_FLAGS)
            if (ov["flags"] & WALK_FLAGS) == oracle.FLAG_NEAR_ACCEPT:
                # exempt only by the accept margin: is the walk inside a ten times narrower band too?  If not, it sits
                # in [1e-7, 1e-6): count it, and count whether the two sides disagree there
                o6 = orc.verify_tree(c["U"][b].float().numpy(), Af, Wf,
                                     Zc[int(offc[b]):int(offc[b]) + otrees[b]["n"] + 1].float().numpy(), int(c["anchor"][b]),
                                     otrees[b], T, round_seed, b, accept_margin=1e-7)
                if not (o6["flags"] & oracle.FLAG_NEAR_ACCEPT):
                    stats["accept_band_walks"] = stats.get("accept_band_walks", 0) + 1
                    same = (int(v["acc_len"][b]) == int(o6["acc_len"]) and int(v["bonus_tok"][b]) == int(o6["bonus"]) and
                            v["acc_tok"][b, :int(o6["acc_len"])].tolist() == o6["acc_tok"][:int(o6["acc_len"])].tolist())
                    if not same:
                        stats["accept_band_disagree"] = stats.get("accept_band_disagree", 0) + 1
        if want_edge:
            n = int(otrees[b]["n"])
            ge = v["edge_stat"][b, :n].numpy()
            for i in range(n):
                assert close(ge[i], ov["edge_stat"][i], rtol=2e-5, atol=1e-6), (b, i, ge[i], ov["edge_stat"][i])
    for k in PARITY_TOTALS:
        PARITY_TOTALS[k] += stats.get(k, 0)
    print(f"parity: {stats['trees']} trees ({stats['trees_exempt']} exempt), {stats['walks']} walks ({stats['walks_exempt']} exempt), "
          f"{stats.get('accept_band_walks', 0)} walks with |u - rho| in [1e-7, 1e-6) ({stats.get('accept_band_disagree', 0)} disagree)")
    return stats
