"""GPU parity of ts_emit_attention_inputs (Section 3.2 item 3) against the CPU oracle, bit for bit.  The
kernel expands the ancestor bitmasks; the oracle walks the parent pointers."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import attention_inputs as att
from gpu_harness import Round, make_gpu, to_cpu
from paper_2609_22098_b200 import synth
from paper_2609_22098_b200.binding import TreeSparkError

pytestmark = pytest.mark.gpu


def small(name, **kw):
    return dataclasses.replace(synth.WORKLOADS[name], **kw)


@pytest.mark.parametrize("name,kw,theta,with_base", [
    ("serve32", dict(V=12000 + 8, B=32), 0.004, True),     # Nmax = 64: 65 rows, one mask word
    ("serve32", dict(V=12000 + 8, B=32), 0.5, False),      # small and empty trees
    ("wide", dict(V=9000, B=8), 0.002, True),              # Nmax = 256: 257 rows, four mask words
    ("decode", dict(V=8000), 0.02, False),
    ("tiny", dict(V=3000, B=3), 0.0, True),                # Nmax = 16, fp32 inputs
])
def test_attention_inputs_match_oracle(name, kw, theta, with_base):
    wl = small(name, **kw)
    rnd = Round(wl, seed=83)
    rnd.theta.fill_(theta)
    ts = make_gpu(wl, rnd.table, max_batch=rnd.B)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 1.0, 91)
    base = torch.randint(0, 5000, (rnd.B,), dtype=torch.int32).cuda() if with_base else None
    out = to_cpu(ts.emit_attention_inputs(rnd.anchor, tree, base))
    torch.cuda.synchronize()
    g = to_cpu(tree)
    assert int(g["n_nodes"].max()) > 0 or theta >= 0.5
    for b in range(rnd.B):
        flat, pos, m = att.attention_inputs(wl.Nmax, int(rnd.anchor[b]), int(base[b]) if with_base else 0,
                                            int(g["n_nodes"][b]), g["tok"][b].numpy(), g["parent"][b].numpy(),
                                            g["depth"][b].numpy())
        assert np.array_equal(out["flat_tok"][b].numpy(), flat), b
        assert np.array_equal(out["pos_ids"][b].numpy(), pos), b
        assert np.array_equal(out["dense_mask"][b].numpy().view(np.int32), m.view(np.int32)), b


def test_outputs_are_optional_and_errors_launch_nothing():
    wl = small("tiny", V=2000, B=2)
    rnd = Round(wl, seed=85)
    ts = make_gpu(wl, rnd.table, max_batch=2)
    tree = ts.expand_tree(rnd.U, rnd.A, rnd.W, rnd.anchor, rnd.theta, 0.0, 3)
    full = ts.emit_attention_inputs(rnd.anchor, tree)
    only = dict(pos_ids=torch.full_like(full["pos_ids"], -7))
    ts.emit_attention_inputs(rnd.anchor, tree, out=only)
    torch.cuda.synchronize()
    assert torch.equal(only["pos_ids"], full["pos_ids"])
    with pytest.raises(TreeSparkError):
        ts.emit_attention_inputs(rnd.anchor, tree, out={"unused": None})
