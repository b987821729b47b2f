"""Glue that drives workload phases through the C ABI on one GPU (marshalling only).

Used by the GPU tests, the smoke check and the benchmark.  torch provides device memory and
streams; every computation happens inside the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np
import torch

from . import binding as B
from . import workloads as W


def to_device(x32: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """float32 numpy values (already storage-rounded) -> device tensor of the storage dtype."""
    if dtype == "bf16":
        bits = W.bf16_bits(x32).view(np.int16)
        return torch.from_numpy(bits).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x32, dtype=np.float32)).to(device)


def to_host_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def torch_dtype(dtype: str):
    return torch.bfloat16 if dtype == "bf16" else torch.float32


class LayerCache:
    """K and V pools of one attention layer (opaque tile format, see ``aspd.h``).

    Each pool sits between two guard pages filled with a byte pattern that no kernel may touch;
    ``canaries_intact()`` tells whether they still hold it (a write one page before or behind a
    pool shows there)."""

    CANARY = 0xA5

    def __init__(self, shape: B.Shape, n_pool_pages: int, device="cuda"):
        nbytes = B.pool_bytes(shape, n_pool_pages)
        if nbytes == 0 and n_pool_pages > 0:
            raise B.AspdError(-3, "aspd_pool_bytes")
        self._guard = max(B.pool_bytes(shape, 1), 256)
        self._raw = []
        for name in ("k", "v"):
            raw = torch.full((self._guard * 2 + max(nbytes, 16),), self.CANARY, dtype=torch.uint8, device=device)
            pool = raw[self._guard: self._guard + max(nbytes, 16)]
            pool.zero_()
            self._raw.append(raw)
            setattr(self, name, pool)

    def canaries_intact(self) -> bool:
        g = self._guard
        return all(bool((raw[:g] == self.CANARY).all()) and bool((raw[-g:] == self.CANARY).all()) for raw in self._raw)


class WorkloadRun:
    """Runs the phases of a workload through kv_append + attention, keeping compared outputs."""

    def __init__(self, wl: W.Workload, kernel: int = B.KERNEL_AUTO, chunk_tokens: int = 0, n_ctas: int = 0,
                 device="cuda", fused: bool = False, stable_cache: bool = False, mask: int = B.MASK_BRANCH_INVISIBLE,
                 combine: int = B.COMBINE_AUTO, wide_rows: int = 0, mma_m: int = 0):
        self.wl, self.kernel, self.chunk_tokens, self.n_ctas, self.device = wl, kernel, chunk_tokens, n_ctas, device
        self.mask = mask            # attention mask of the parallel steps (ASPD_MASK_*)
        self.combine = combine      # where the split-K records are merged (ASPD_COMBINE_*)
        self.wide_rows = wide_rows  # rows of a row block in plans that deal whole streams (0 = automatic)
        self.mma_m = mma_m          # M of the tensor-core kernel's MMAs in stream-K plans (0 = automatic)
        self.stable_cache = stable_cache
        self.fused = fused          # attention phases go through aspd_branch_step / aspd_serial_step
        self.shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
        self.cache = LayerCache(self.shape, wl.n_pool_pages, device)
        self.outputs: List[np.ndarray] = []
        self.positions = []
        self.plans = []

    def step(self, ph: W.Phase, attend: bool = True, keep_plan: bool = False, pos_override=None) -> Optional[np.ndarray]:
        """pos_override: caller-given position IDs of the phase's new tokens (a position-ID variant):
        passed to aspd_kv_append and, as q_pos, to the plan."""
        wl = self.wl
        plan = B.Plan(self.shape, ph.desc, wl.n_pool_pages, ph.mode, q_pos=pos_override, kernel=self.kernel,
                      chunk_tokens=self.chunk_tokens, n_ctas=self.n_ctas, stable_cache=self.stable_cache, mask=self.mask,
                      combine=self.combine, wide_rows=self.wide_rows, mma_m=self.mma_m)
        pos, slot, req = B.positions(ph.desc, ph.mode)
        if pos_override is not None:
            pos = np.ascontiguousarray(pos_override, dtype=np.int32)
        self.positions.append((pos, slot, req))
        out = None
        if plan.n_new > 0:
            pos_d = torch.from_numpy(pos.copy()).to(self.device)
            k_d, v_d = to_device(ph.k_new, wl.dtype, self.device), to_device(ph.v_new, wl.dtype, self.device)
            do_attn = attend and ph.q is not None
            if do_attn and self.fused:
                q_d = to_device(ph.q, wl.dtype, self.device)
                out_d = torch.empty_like(q_d)
                (B.branch_step if ph.mode == W.MODE_BRANCH else B.serial_step)(plan, q_d, k_d, v_d, self.cache.k,
                                                                               self.cache.v, out_d)
            else:
                B.kv_append(plan, k_d, v_d, pos_d, self.cache.k, self.cache.v)
            if do_attn:
                if not self.fused:
                    q_d = to_device(ph.q, wl.dtype, self.device)
                    out_d = torch.empty_like(q_d)
                    (B.branch_attn if ph.mode == W.MODE_BRANCH else B.serial_attn)(plan, q_d, self.cache.k, self.cache.v, out_d)
                torch.cuda.synchronize()
                st = plan.status()
                if st != 0:
                    raise B.AspdError(st, "device status")
                out = to_host_f32(out_d)
                if ph.compare:
                    self.outputs.append(out)
        if keep_plan:
            self.plans.append(plan)
        else:
            torch.cuda.synchronize()
            plan.destroy()
        return out

    def read_token(self, pool: str, page: int, row: int, head: int) -> np.ndarray:
        return B.debug_read_token(self.shape, self.cache.k if pool == "k" else self.cache.v, page, row, head)


def run_workload(wl: W.Workload, **kw) -> WorkloadRun:
    run = WorkloadRun(wl, **kw)
    for ph in wl.phases:
        run.step(ph)
    return run
