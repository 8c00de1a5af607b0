"""ts_score_parents_static: the scoring call for callers that cannot give the library a workspace
(no device memory left to hand out, or no permission to allocate on the request path).  Its scratch
is an array built into the library, shared by every call on the device, so the checks here are that
it returns what the workspace version returns, twice in a row with different parent lists (the
second call must not see anything of the first), and that it refuses what does not fit.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import dataclasses

import pytest
import torch

from gpu_harness import Round, close, make_gpu, to_cpu
from paper_2609_22098_b200 import synth
from paper_2609_22098_b200.binding import TreeSparkError

pytestmark = pytest.mark.gpu


def parent_list(P, B, D, V, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randint(0, B, (P,), generator=g, dtype=torch.int32).cuda(),
            torch.randint(0, D, (P,), generator=g, dtype=torch.int32).cuda(),
            torch.randint(0, V, (P,), generator=g, dtype=torch.int32).cuda(),
            torch.randint(0, 2 ** 62, (P,), generator=g, dtype=torch.int64).cuda())


def same(a, b, K):
    a, b = to_cpu(a), to_cpu(b)
    assert torch.equal(a["top_tok"], b["top_tok"]) and torch.equal(a["draw_tok"], b["draw_tok"])
    for name in ("lse0", "lseT", "top_logit", "draw_logit"):
        x, y = a[name].reshape(-1), b[name].reshape(-1)
        assert all(close(x[i], y[i]) for i in range(x.numel())), name


@pytest.mark.parametrize("T", [0.0, 1.0])
def test_static_scratch_scoring_matches_workspace_scoring_twice(T):
    wl = dataclasses.replace(synth.WORKLOADS["serve32"], V=30000 + 16, B=4)
    rnd = Round(wl, seed=5)
    ts = make_gpu(wl, rnd.table, max_batch=4)
    for call, P in enumerate((37, 9)):          # second call is smaller: stale records must not leak
        req, dep, tok, hsh = parent_list(P, 4, wl.D, wl.V, seed=100 + call)
        want = ts.score_parents(rnd.U, rnd.A, rnd.W, req, dep, tok, hsh, T, seed=31 + call)
        got = ts.score_parents_static(rnd.U, rnd.A, rnd.W, req, dep, tok, hsh, T, seed=31 + call,
                                      out=ts.alloc_score_outputs(P))
        torch.cuda.synchronize()
        same(got, want, wl.K)


def test_static_scratch_refuses_what_does_not_fit():
    wl = dataclasses.replace(synth.WORKLOADS["serve32"], V=30000 + 16, B=64)
    rnd = Round(wl, seed=6, B=2)
    ts = make_gpu(wl, rnd.table, max_batch=64)
    P = 4000                                    # far beyond 8 MiB of records for this tiling
    req, dep, tok, hsh = parent_list(P, 2, wl.D, wl.V, seed=1)
    with pytest.raises(TreeSparkError, match="built-in array"):
        ts.score_parents_static(rnd.U, rnd.A, rnd.W, req, dep, tok, hsh, 1.0, seed=1, out=ts.alloc_score_outputs(P))
