"""Thin Python binding of the C ABI in ``include/aspd.h`` (argument marshalling only).

Every step of the path runs in the CUDA library; nothing here computes.  Descriptors are
given as a dict of int32 numpy arrays (struct of arrays, the form the workload generator
emits) and packed into the C structs.  Device buffers are torch tensors (or anything with
``data_ptr()``), host buffers numpy arrays.  There is no CPU fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import numpy as np

from . import build as _build

MODE_BRANCH, MODE_SERIAL = 0, 1
DTYPE_F32, DTYPE_BF16 = 0, 1
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_MMA = 0, 1, 2
Q_SHARED = -1
POS_AUTO = -1
MASK_BRANCH_INVISIBLE, MASK_SHARED = 0, 1
COMBINE_AUTO, COMBINE_KERNEL, COMBINE_FUSED = 0, 1, 2

REQUEST_DTYPE = np.dtype([(n, np.int32) for n in
                          ("prefix_len", "n_branches", "branch_begin", "page_begin", "n_pages", "tail_off", "tail_len")])
BRANCH_DTYPE = np.dtype([(n, np.int32) for n in ("kv_off", "kv_len", "pos_start", "q_len")])
ITEM_DTYPE = np.dtype([(n, np.int32) for n in
                       ("q_tok0", "n_q_tok", "kv_head", "page0", "n_pages", "key0", "part_slot", "request", "row_block",
                        "n_parts")])


class Shape(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("dtype", ctypes.c_int32), ("rope_theta", ctypes.c_float),
                ("sm_scale", ctypes.c_float)]


class Tuning(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("chunk_tokens", ctypes.c_int32), ("n_ctas", ctypes.c_int32),
                ("host_only", ctypes.c_int32), ("stable_cache", ctypes.c_int32), ("mask", ctypes.c_int32),
                ("updatable", ctypes.c_int32), ("combine", ctypes.c_int32), ("wide_rows", ctypes.c_int32),
                ("mma_m", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("n_new", ctypes.c_int32), ("n_items", ctypes.c_int32), ("n_partials", ctypes.c_int32),
                ("n_stream_pages", ctypes.c_int32), ("kernel", ctypes.c_int32), ("chunk_tokens", ctypes.c_int32),
                ("n_ctas", ctypes.c_int32), ("fused_append", ctypes.c_int32),
                ("direct_output", ctypes.c_int32), ("max_rows_per_item", ctypes.c_int32),
                ("dealt", ctypes.c_int32), ("single_launch", ctypes.c_int32), ("mma_m", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("workspace_bytes", ctypes.c_int64), ("kv_tokens_read", ctypes.c_int64),
                ("algorithmic_bytes", ctypes.c_int64)]


class AspdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


EXPORTS = ("aspd_strerror", "aspd_pool_bytes", "aspd_count_new_tokens", "aspd_positions", "aspd_visible_slots",
           "aspd_visible_slots_masked", "aspd_plan_create", "aspd_plan_update", "aspd_plan_destroy", "aspd_release_cached_memory", "aspd_plan_info", "aspd_plan_items", "aspd_plan_cta_ranges", "aspd_plan_stream_pages",
           "aspd_plan_token_ranges", "aspd_plan_shared_mask_tables", "aspd_plan_status",
           "aspd_kv_append", "aspd_branch_attn", "aspd_serial_attn", "aspd_attn_partials", "aspd_attn_combine", "aspd_step_partials",
           "aspd_branch_step", "aspd_serial_step", "aspd_step_host", "aspd_step_host_async", "aspd_attn_static", "aspd_static_status", "aspd_k_rerotate", "aspd_k_rerotate_ranges", "aspd_k_rerotate_ranges_layers", "aspd_debug_read_token", "aspd_debug_bounded_wait", "aspd_debug_profile", "aspd_debug_pool_limit")

_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load the CUDA library (building it first if the sources are newer).  Fails loudly."""
    global _lib
    if _lib is None:
        # ASPD_LIBRARY selects another build of the same sources: the GPU tests run a subset once
        # more against the -DASPD_DEBUG_BOUNDS build (kernels that check page ids and rows) this way
        path = os.environ.get("ASPD_LIBRARY") or _build.build()
        L = ctypes.CDLL(path)
        L.aspd_strerror.restype = ctypes.c_char_p
        L.aspd_strerror.argtypes = [ctypes.c_int]
        L.aspd_pool_bytes.restype = ctypes.c_size_t
        L.aspd_pool_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int64]
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.aspd_count_new_tokens.argtypes = [vp, vp, ci, ci]
        L.aspd_positions.argtypes = [vp, vp, ci, ci, vp, vp, vp]
        L.aspd_visible_slots.argtypes = [vp, vp, ci, ci, ci, vp]
        L.aspd_visible_slots_masked.argtypes = [vp, vp, ci, ci, ci, ci, vp]
        L.aspd_plan_create.argtypes = [vp, vp, vp, vp, ci, ctypes.c_int64, ci, vp, vp, vp, vp]
        L.aspd_plan_destroy.argtypes = [vp]
        L.aspd_plan_update.argtypes = [vp, vp, vp, vp, ci, vp, vp]
        L.aspd_release_cached_memory.argtypes = []
        L.aspd_plan_info.argtypes = [vp, vp]
        L.aspd_plan_items.argtypes = [vp, vp, ci]
        L.aspd_plan_cta_ranges.argtypes = [vp, vp, ci]
        L.aspd_plan_stream_pages.argtypes = [vp, vp, vp, ci]
        L.aspd_plan_token_ranges.argtypes = [vp, vp, vp, vp, ci]
        L.aspd_plan_shared_mask_tables.argtypes = [vp, vp, vp]
        L.aspd_plan_status.argtypes = [vp, vp]
        L.aspd_kv_append.argtypes = [vp] * 7
        L.aspd_branch_attn.argtypes = [vp] * 6
        L.aspd_serial_attn.argtypes = [vp] * 6
        L.aspd_attn_partials.argtypes = [vp] * 5
        L.aspd_attn_combine.argtypes = [vp] * 3
        L.aspd_step_partials.argtypes = [vp] * 7
        L.aspd_branch_step.argtypes = [vp] * 8
        L.aspd_serial_step.argtypes = [vp] * 8
        L.aspd_step_host.argtypes = [vp] * 9
        L.aspd_step_host_async.argtypes = [vp] * 9
        L.aspd_attn_static.argtypes = [vp] * 6
        L.aspd_static_status.argtypes = [vp]
        L.aspd_k_rerotate.argtypes = [vp, vp, vp, vp, vp, ci, vp]
        L.aspd_k_rerotate_ranges.argtypes = [vp, vp, vp, vp, ci, vp]
        L.aspd_k_rerotate_ranges_layers.argtypes = [vp, vp, ci, vp, vp, ci, vp]
        L.aspd_debug_bounded_wait.argtypes = [ctypes.c_int64, vp, vp]
        L.aspd_debug_profile.argtypes = [vp, ci]
        L.aspd_debug_pool_limit.argtypes = [vp, ctypes.c_int64]
        L.aspd_debug_read_token.argtypes = [vp, vp, ctypes.c_int64, ci, ci, vp, vp]
        for name in EXPORTS:
            if name not in ("aspd_strerror", "aspd_pool_bytes"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().aspd_strerror(int(status)).decode()


def _check(rc: int, where: str) -> int:
    if rc < 0:
        raise AspdError(rc, where)
    return rc


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, np.ndarray):
        assert x.flags.c_contiguous
        return x.ctypes.data
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return getattr(stream, "cuda_stream", stream)


def make_shape(n_q_heads, n_kv_heads, head_dim, page_size, dtype, rope_theta, sm_scale) -> Shape:
    code = {"f32": DTYPE_F32, "bf16": DTYPE_BF16}.get(dtype, dtype)
    return Shape(n_q_heads, n_kv_heads, head_dim, page_size, code, rope_theta, sm_scale)


def pack_descriptors(desc: Dict[str, np.ndarray]):
    """dict of int32 arrays -> (aspd_request_t[], aspd_branch_t[], page_ids) numpy arrays.

    A missing ``br_pos_start`` becomes ``ASPD_POS_AUTO``: the library then derives the paper's shared
    position-ID rule (Eq. 4: stage_start) itself."""
    n_req = len(desc["prefix_len"])
    req = np.zeros(n_req, dtype=REQUEST_DTYPE)
    for name in REQUEST_DTYPE.names:
        req[name] = desc[name]
    n_br = len(desc["br_kv_off"])
    br = np.zeros(n_br, dtype=BRANCH_DTYPE)
    br["kv_off"], br["kv_len"], br["q_len"] = desc["br_kv_off"], desc["br_kv_len"], desc["br_q_len"]
    br["pos_start"] = desc["br_pos_start"] if "br_pos_start" in desc else POS_AUTO
    pages = np.ascontiguousarray(desc["page_ids"], dtype=np.int32)
    return req, br, pages


def pool_bytes(shape: Shape, n_pages: int) -> int:
    return int(lib().aspd_pool_bytes(ctypes.addressof(shape), n_pages))


def count_new_tokens(desc, mode: int) -> int:
    req, br, _ = pack_descriptors(desc)
    return _check(lib().aspd_count_new_tokens(_ptr(req), _ptr(br), len(req), mode), "aspd_count_new_tokens")


def positions(desc, mode: int):
    """(pos, slot, request) int32 arrays of the step's new tokens (host integer code in the library)."""
    req, br, _ = pack_descriptors(desc)
    n = _check(lib().aspd_count_new_tokens(_ptr(req), _ptr(br), len(req), mode), "aspd_count_new_tokens")
    pos, slot, rq = (np.zeros(max(n, 1), dtype=np.int32) for _ in range(3))
    _check(lib().aspd_positions(_ptr(req), _ptr(br), len(req), mode, _ptr(pos), _ptr(slot), _ptr(rq)), "aspd_positions")
    return pos[:n], slot[:n], rq[:n]


def visible_slots(desc, mode: int, n_slots: int, mask: int = 0) -> np.ndarray:
    req, br, _ = pack_descriptors(desc)
    n = _check(lib().aspd_count_new_tokens(_ptr(req), _ptr(br), len(req), mode), "aspd_count_new_tokens")
    vis = np.zeros((max(n, 1), n_slots), dtype=np.uint8)
    if mask == MASK_BRANCH_INVISIBLE:
        _check(lib().aspd_visible_slots(_ptr(req), _ptr(br), len(req), mode, n_slots, _ptr(vis)), "aspd_visible_slots")
    else:
        _check(lib().aspd_visible_slots_masked(_ptr(req), _ptr(br), len(req), mode, mask, n_slots, _ptr(vis)),
               "aspd_visible_slots_masked")
    return vis[:n]


class Plan:
    """Owner of an ``aspd_plan_t`` (see ``aspd_plan_create``)."""

    def __init__(self, shape: Shape, desc, n_pool_pages: int, mode: int, q_pos=None, kernel: int = KERNEL_AUTO,
                 chunk_tokens: int = 0, n_ctas: int = 0, host_only: bool = False, stable_cache: bool = False, stream=None,
                 mask: int = 0, updatable: bool = False, combine: int = COMBINE_AUTO, wide_rows: int = 0, mma_m: int = 0):
        self.shape, self.mode = shape, mode
        req, br, pages = pack_descriptors(desc)
        tune = Tuning(kernel, chunk_tokens, n_ctas, 1 if host_only else 0, 1 if stable_cache else 0, mask, 1 if updatable else 0, combine, wide_rows, mma_m)
        qp = None if q_pos is None else np.ascontiguousarray(q_pos, dtype=np.int32)
        handle = ctypes.c_void_p()
        self._h = None
        _check(lib().aspd_plan_create(ctypes.addressof(shape), _ptr(req), _ptr(br), _ptr(pages), len(req), n_pool_pages,
                                      mode, _ptr(qp), ctypes.addressof(tune), None if host_only else _stream(stream),
                                      ctypes.addressof(handle)), "aspd_plan_create")
        self._h = handle
        self.info = PlanInfo()
        _check(lib().aspd_plan_info(self._h, ctypes.addressof(self.info)), "aspd_plan_info")
        self.n_new = self.info.n_new

    def update(self, desc, q_pos=None, stream=None) -> None:
        """Re-plan in place for the next step of the same batch (see ``aspd_plan_update``)."""
        req, br, pages = pack_descriptors(desc)
        qp = None if q_pos is None else np.ascontiguousarray(q_pos, dtype=np.int32)
        _check(lib().aspd_plan_update(self._h, _ptr(req), _ptr(br), _ptr(pages), len(req), _ptr(qp), _stream(stream)),
               "aspd_plan_update")
        _check(lib().aspd_plan_info(self._h, ctypes.addressof(self.info)), "aspd_plan_info")

    def items(self) -> np.ndarray:
        items = np.zeros(max(self.info.n_items, 1), dtype=ITEM_DTYPE)
        _check(lib().aspd_plan_items(self._h, _ptr(items), self.info.n_items), "aspd_plan_items")
        return items[: self.info.n_items]

    def cta_ranges(self) -> np.ndarray:
        """first[c] .. first[c + 1]: the items CTA c of the persistent grid owns."""
        first = np.zeros(self.info.n_ctas + 1, np.int32)
        _check(lib().aspd_plan_cta_ranges(self._h, _ptr(first), len(first)), "aspd_plan_cta_ranges")
        return first

    def stream_pages(self):
        """(physical page, valid rows) of every page the step reads, as two int32 arrays."""
        n = self.info.n_stream_pages
        ids, nv = np.zeros(max(n, 1), np.int32), np.zeros(max(n, 1), np.int32)
        _check(lib().aspd_plan_stream_pages(self._h, _ptr(ids), _ptr(nv), n), "aspd_plan_stream_pages")
        return ids[:n], nv[:n]

    def token_ranges(self):
        """(pe, lo, hi) per new token: it may attend stream keys [0, pe) and [lo, hi)."""
        n = self.n_new
        pe, lo, hi = (np.zeros(max(n, 1), np.int32) for _ in range(3))
        _check(lib().aspd_plan_token_ranges(self._h, _ptr(pe), _ptr(lo), _ptr(hi), n), "aspd_plan_token_ranges")
        return pe[:n], lo[:n], hi[:n]

    def shared_mask_tables(self):
        """(below per new token, page index in its branch per stream page) of a MASK_SHARED plan."""
        below = np.zeros(max(self.n_new, 1), np.int32)
        pib = np.zeros(max(self.info.n_stream_pages, 1), np.int32)
        _check(lib().aspd_plan_shared_mask_tables(self._h, _ptr(below), _ptr(pib)), "aspd_plan_shared_mask_tables")
        return below[: self.n_new], pib[: self.info.n_stream_pages]

    def status(self, stream=None) -> int:
        return lib().aspd_plan_status(self._h, _stream(stream))

    def destroy(self):
        if self._h is not None:
            lib().aspd_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def kv_append(plan: Plan, k_new, v_new, pos, k_pool, v_pool, stream=None) -> None:
    _check(lib().aspd_kv_append(plan._h, _ptr(k_new), _ptr(v_new), _ptr(pos), _ptr(k_pool), _ptr(v_pool), _stream(stream)),
           "aspd_kv_append")


def branch_attn(plan: Plan, q, k_pool, v_pool, out, stream=None) -> None:
    _check(lib().aspd_branch_attn(plan._h, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(out), _stream(stream)),
           "aspd_branch_attn")


def serial_attn(plan: Plan, q, k_pool, v_pool, out, stream=None) -> None:
    _check(lib().aspd_serial_attn(plan._h, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(out), _stream(stream)),
           "aspd_serial_attn")


def attn_partials(plan: Plan, q, k_pool, v_pool, stream=None) -> None:
    _check(lib().aspd_attn_partials(plan._h, _ptr(q), _ptr(k_pool), _ptr(v_pool), _stream(stream)), "aspd_attn_partials")


def attn_combine(plan: Plan, out, stream=None) -> None:
    _check(lib().aspd_attn_combine(plan._h, _ptr(out), _stream(stream)), "aspd_attn_combine")


def step_partials(plan: Plan, q, k_new, v_new, k_pool, v_pool, stream=None) -> None:
    _check(lib().aspd_step_partials(plan._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _stream(stream)),
           "aspd_step_partials")


def branch_step(plan: Plan, q, k_new, v_new, k_pool, v_pool, out, stream=None) -> None:
    _check(lib().aspd_branch_step(plan._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(out),
                                  _stream(stream)), "aspd_branch_step")


def serial_step(plan: Plan, q, k_new, v_new, k_pool, v_pool, out, stream=None) -> None:
    _check(lib().aspd_serial_step(plan._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool), _ptr(out),
                                  _stream(stream)), "aspd_serial_step")


def step_host(plan: Plan, q, k_new, v_new, pos, k_pool, v_pool, out, stream=None) -> None:
    """Whole step from host (numpy / pinned torch CPU) buffers; ``out`` is a host buffer."""
    _check(lib().aspd_step_host(plan._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(pos), _ptr(k_pool), _ptr(v_pool),
                                _ptr(out), _stream(stream)), "aspd_step_host")


def release_cached_memory() -> None:
    """Free the device blocks of destroyed plans that the library keeps for reuse."""
    _check(lib().aspd_release_cached_memory(), "aspd_release_cached_memory")


def step_host_async(plan: Plan, q, k_new, v_new, pos, k_pool, v_pool, out, stream=None) -> None:
    """``step_host`` without the final synchronisation (pinned host buffers; see ``aspd_step_host_async``)."""
    _check(lib().aspd_step_host_async(plan._h, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(pos), _ptr(k_pool), _ptr(v_pool),
                                      _ptr(out), _stream(stream)), "aspd_step_host_async")


def k_rerotate(shape: Shape, k_pool, pages, rows, delta, stream=None) -> None:
    """Rotate cached keys by ``delta`` positions in place (device int32 arrays of equal length)."""
    _check(lib().aspd_k_rerotate(ctypes.addressof(shape), _ptr(k_pool), _ptr(pages), _ptr(rows), _ptr(delta), int(pages.numel()),
                                 _stream(stream)), "aspd_k_rerotate")


def k_rerotate_ranges(shape: Shape, k_pool, page_table, ranges, stream=None) -> None:
    """Rotate whole slot ranges in place: ``ranges`` is a host int32 array [n][4] of (page-table
    base, first slot, count, delta), ``page_table`` the device int32 page tables."""
    ranges = np.ascontiguousarray(ranges, dtype=np.int32).reshape(-1, 4)
    _check(lib().aspd_k_rerotate_ranges(ctypes.addressof(shape), _ptr(k_pool), _ptr(page_table), _ptr(ranges), len(ranges),
                                        _stream(stream)), "aspd_k_rerotate_ranges")


def k_rerotate_ranges_layers(shape: Shape, k_pools, page_table, ranges, stream=None) -> None:
    """The same for the K pools of several layers (a sequence of device tensors) in one launch."""
    ranges = np.ascontiguousarray(ranges, dtype=np.int32).reshape(-1, 4)
    ptrs = (ctypes.c_void_p * len(k_pools))(*[_ptr(k) for k in k_pools])
    _check(lib().aspd_k_rerotate_ranges_layers(ctypes.addressof(shape), ptrs, len(k_pools), _ptr(page_table), _ptr(ranges),
                                               len(ranges), _stream(stream)), "aspd_k_rerotate_ranges_layers")


def debug_bounded_wait(limit_cycles: int, stream=None) -> int:
    """Status a bounded device-side wait reports when nothing ever satisfies it (ASPD_ERR_TIMEOUT)."""
    st = np.zeros(1, dtype=np.int32)
    _check(lib().aspd_debug_bounded_wait(int(limit_cycles), _ptr(st), _stream(stream)), "aspd_debug_bounded_wait")
    return int(st[0])


STATIC_SCRATCH_BYTES = 8 << 20


def attn_static(plan: Plan, q, k_pool, v_pool, out, stream=None) -> None:
    """Attention of a step for callers that cannot allocate device memory: ``plan`` is a
    host-only plan and all scratch lives in an array compiled into the library (see
    ``aspd_attn_static`` in ``aspd.h`` for the size limit and the sharing rules)."""
    _check(lib().aspd_attn_static(plan._h, _ptr(q), _ptr(k_pool), _ptr(v_pool), _ptr(out), _stream(stream)),
           "aspd_attn_static")


def static_status(stream=None) -> int:
    """Status word of the last ``attn_static`` call on the current device (synchronises the stream)."""
    return lib().aspd_static_status(_stream(stream))


def debug_pool_limit(plan: Plan, n_pages: int) -> int:
    """Lower the page count a checking build's kernels compare page ids against (status; -3 in an
    ordinary build)."""
    return lib().aspd_debug_pool_limit(plan._h, int(n_pages))


def debug_profile(device_buf, cta: int = 0) -> int:
    """Point the profiling build's stamps at ``device_buf`` (int64 device tensor); returns the
    status (ASPD_ERR_UNSUPPORTED = -3 in an ordinary build)."""
    return lib().aspd_debug_profile(_ptr(device_buf), cta)


def debug_read_token(shape: Shape, pool, page: int, row: int, kv_head: int, stream=None) -> np.ndarray:
    out = np.zeros(shape.head_dim, dtype=np.float32)
    _check(lib().aspd_debug_read_token(ctypes.addressof(shape), _ptr(pool), page, row, kv_head, _ptr(out), _stream(stream)),
           "aspd_debug_read_token")
    return out
