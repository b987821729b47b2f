"""The checking build of the library (-DASPD_DEBUG_BOUNDS): kernels that compare every page id and
row they are about to use with the pool's size, record ASPD_ERR_BAD_DESCRIPTOR in the plan's status
word on a violation and leave the access out.  Nothing here goes out of bounds, faults or traps: the
violation is made by LOWERING the limit the kernels compare against, while the pools keep their size.

A process loads one build of the library, so each case runs in a child process with ASPD_LIBRARY
pointing at the checking build.
"""
import os
import subprocess
import sys

import pytest

from paper_2508_08895_b200 import binding as B, build as build_mod, workloads as W

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _child_env():
    env = dict(os.environ)
    env["ASPD_LIBRARY"] = build_mod.build_debug_bounds()
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    return env


def test_parity_subset_is_green_on_the_checking_build():
    """The same parity cases through kernels that check: the same outcomes and a clean status word
    (the engine raises on a non-zero status after every step)."""
    sel = "config2 or ragged_edges or second_parallel_stage or shared_mask_variant or fused_step_appends or config4"
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-x", "-q", "-m", "gpu",
                          "-k", sel], env=_child_env(), capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout and "failed" not in res.stdout


CHILD = r"""
import numpy as np, torch
from paper_2508_08895_b200 import binding as B, engine as E, workloads as W
from oracle.run import run_workload as oracle_run
for kernel in (B.KERNEL_AUTO, B.KERNEL_GENERIC):
    for fused in (False, True):
        wl = W.build_segment_workload("lim", 41, 28, 4, 128, "bf16", 1e6, [300], [[40, 17, 129]], [[1, 1, 1]])
        run = E.WorkloadRun(wl, kernel=kernel)
        for ph in wl.phases[:-1]:
            run.step(ph)
        ph = wl.phases[-1]
        pos, _, _ = B.positions(ph.desc, ph.mode)
        q, k, v = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
        pos_d = torch.from_numpy(pos.copy()).cuda()
        out = torch.zeros_like(q)
        # a lowered limit: most page ids of the step are now "outside"; the kernels flag and skip
        plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, kernel=kernel)
        assert B.debug_pool_limit(plan, wl.n_pool_pages + 1) == -1          # never beyond the real size
        assert B.debug_pool_limit(plan, 1) == 0
        if fused:
            B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, out)
        else:
            B.kv_append(plan, k, v, pos_d, run.cache.k, run.cache.v)
            B.branch_attn(plan, q, run.cache.k, run.cache.v, out)
        torch.cuda.synchronize()
        assert plan.status() == -2, plan.status()
        assert run.cache.canaries_intact()
        plan.destroy()
        # the context is as usable as before: a fresh plan with the true limit is clean and right
        plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, kernel=kernel)
        B.kv_append(plan, k, v, pos_d, run.cache.k, run.cache.v)
        B.branch_attn(plan, q, run.cache.k, run.cache.v, out)
        torch.cuda.synchronize()
        assert plan.status() == 0
        err = np.abs(out.float().cpu().numpy().astype(np.float64) - oracle_run(wl).outputs[-1])
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
        plan.destroy()
print("CHILD-OK")
"""


def test_a_page_beyond_the_limit_is_flagged_and_skipped():
    res = subprocess.run([sys.executable, "-c", CHILD], env=_child_env(), capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0 and "CHILD-OK" in res.stdout, res.stdout[-2000:] + res.stderr[-3000:]


def test_the_product_build_has_no_such_check():
    wl = W.build_segment_workload("lim", 41, 28, 4, 128, "bf16", 1e6, [30], [[4]], [[1]])
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    plan = B.Plan(shape, wl.phases[-1].desc, wl.n_pool_pages, wl.phases[-1].mode)
    assert B.debug_pool_limit(plan, 1) == -3
    plan.destroy()
