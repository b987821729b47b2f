"""Drive a whole synthetic workload through the fp64 oracle -- TEST INFRASTRUCTURE ONLY.

Executes the phases of a workload (cache fill, parallel step, serial steps) with the oracle's
own position rule, paged append and attention, and returns what the CUDA path is compared
against.  Imports nothing from the CUDA library or its binding.
"""
from __future__ import annotations

import numpy as np

import oracle


class OracleRun:
    def __init__(self, wl, mask=oracle.MASK_BRANCH_INVISIBLE):
        self.wl = wl
        self.mask = mask       # attention mask of the parallel steps (the ablation's visible mask: MASK_SHARED)
        self.k_pool, self.v_pool = oracle.make_pools(wl.n_pool_pages, wl.Hkv, wl.page_size, wl.d)
        self.outputs = []      # one [n_new][Hq][d] array per compared phase
        self.positions = []    # per phase: (pos, slot, req) int32 arrays

    def step(self, ph, attend=True, pos_override=None):
        """pos_override: position IDs of a position-ID variant for this phase's new tokens (keys
        and queries); default: the paper's rule (Eq. 4)."""
        wl = self.wl
        pos, slot, req = oracle.new_tokens(ph.desc, ph.mode)
        if pos_override is not None:
            pos = np.ascontiguousarray(pos_override, dtype=np.int32)
        self.positions.append((pos, slot, req))
        oracle.kv_append(ph.desc, ph.k_new, ph.v_new, pos, req, slot, self.k_pool, self.v_pool, wl.theta)
        if attend and ph.q is not None:
            out = oracle.attn(ph.desc, ph.mode, ph.q, self.k_pool, self.v_pool, wl.theta, wl.sm_scale,
                              q_pos=pos if pos_override is not None else None, mask=self.mask)
            if ph.compare:
                self.outputs.append(out)
            return out
        return None


def run_workload(wl, mask=oracle.MASK_BRANCH_INVISIBLE) -> OracleRun:
    run = OracleRun(wl, mask)
    for ph in wl.phases:
        run.step(ph)
    return run
