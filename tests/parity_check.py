"""The comparison every GPU parity test applies: the CUDA path's output against the fp64 oracle's.

  bf16 in / fp32 accumulate : max-abs <= 2e-2, mean-abs <= 2e-3 (the acceptance bound) and a relative
                              L2 error <= 1e-2, because with logits ~ N(0, 1) over thousands of keys the
                              outputs themselves are only a few 1e-2 large, so the absolute bound alone
                              would let a wrong kernel through
  fp32                      : max-abs <= 1e-4, mean-abs <= 1e-5, relative L2 <= 1e-5
"""
import numpy as np

TOL = {"bf16": dict(max_abs=2e-2, mean_abs=2e-3, rel_l2=1e-2), "f32": dict(max_abs=1e-4, mean_abs=1e-5, rel_l2=1e-5)}


def errors(gpu, ref):
    """(max-abs, mean-abs, relative L2) of gpu against ref."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(gpu - ref)
    return float(err.max()), float(err.mean()), float(np.linalg.norm(gpu - ref) / max(np.linalg.norm(ref), 1e-30))


def check(gpu, ref, dtype, what="", tol=None):
    gpu = np.asarray(gpu, dtype=np.float64)
    assert gpu.shape == ref.shape, what
    assert np.isfinite(gpu).all(), what
    t = tol or TOL[dtype]
    mx, mean, rel = errors(gpu, ref)
    assert mx <= t["max_abs"], (what, "max-abs", mx)
    assert mean <= t["mean_abs"], (what, "mean-abs", mean)
    assert rel <= t["rel_l2"], (what, "rel-l2", rel)
