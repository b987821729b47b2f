"""Seeded random requests x random plan options against the oracle (GPU).

Every case draws a small batch (decode steps, whole branches in one step, mixtures, a second
parallel stage), a mask (the paper's or the ablation's visible one) and plan options (grid size,
forced cuts, fused or separate append, stable-cache promise, kernel), so that the planner's regimes
(stream-K cuts, dealt whole streams, wide row blocks, records or direct output) meet shapes no
hand-written case lists.  The bounds are those of the other parity tests, the relative-L2 gate included.
"""
import numpy as np
import pytest

from oracle.run import run_workload as oracle_run
from paper_2508_08895_b200 import binding as B, workloads as W
from parity_check import check

pytestmark = pytest.mark.gpu


def draw_case(n):
    rng = np.random.default_rng(7 * 100003 + n)
    style = ["decode", "prefill", "mixed", "twostage"][n % 4]
    if style == "twostage":
        nb = int(rng.integers(1, 4))
        wl = W.build_two_stage_workload("r", 2000 + n, 28, 4, 128, "bf16", 1e6, int(rng.integers(1, 300)),
                                        [int(x) for x in rng.integers(1, 40, size=int(rng.integers(1, 4)))], int(rng.integers(1, 5)),
                                        [int(x) for x in rng.integers(0, 50, size=nb)], [int(x) for x in rng.integers(1, 4, size=nb)],
                                        serial_steps=1)
    else:
        n_req = int(rng.integers(1, 7))
        prefix = [int(x) for x in rng.integers(0, 600, size=n_req)]
        prior, ql = [], []
        for r in range(n_req):
            nb = int(rng.integers(1, 6))
            if style == "decode":
                p, q = rng.integers(0, 150, size=nb), rng.integers(0, 2, size=nb)
            elif style == "prefill":
                p, q = rng.integers(0, 30, size=nb), rng.integers(1, 70, size=nb)
            else:
                p, q = rng.integers(0, 80, size=nb), rng.integers(0, 25, size=nb)
            p, q = [int(x) for x in p], [int(x) for x in q]
            if sum(q) == 0 or (prefix[r] == 0 and p[0] == 0 and q[0] == 0):
                q[0] = 1
            prior.append(p); ql.append(q)
        wl = W.build_segment_workload("r", 2000 + n, 28, 4, 128, "bf16", 1e6, prefix, prior, ql, serial_steps=int(rng.integers(0, 2)))
    kw = dict(n_ctas=int(rng.choice([0, 1, 2, 3, 5, 8, 16, 37])), fused=bool(rng.integers(0, 2)), mask=int(rng.integers(0, 2)),
              stable_cache=bool(rng.integers(0, 2)))
    if rng.integers(0, 4) == 0:
        kw["chunk_tokens"] = int(rng.choice([16, 48, 128, 1024]))
    if rng.integers(0, 6) == 0:
        kw["kernel"] = B.KERNEL_GENERIC
    kw["combine"] = int(np.random.default_rng(991 + n).integers(0, 3))      # drawn apart: the cases above stay what they were
    return wl, kw


@pytest.mark.parametrize("block", range(6))
def test_random_requests_and_plan_options(block):
    from paper_2508_08895_b200 import engine as E
    for n in range(block * 8, block * 8 + 8):
        wl, kw = draw_case(n)
        ref = oracle_run(wl, kw["mask"])
        run = E.run_workload(wl, **kw)
        assert len(run.outputs) == len(ref.outputs) and len(ref.outputs) > 0, (n, kw)
        for g, r in zip(run.outputs, ref.outputs):
            check(g, r, wl.dtype, f"case {n} {kw}")
        assert run.cache.canaries_intact(), (n, kw)
