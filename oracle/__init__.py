"""fp64 CPU oracle of ASPD's branch-isolated attention step -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``aspd_oracle.c`` (the arithmetic lives there, with the
citations).  Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do, and this package imports
nothing from them.

Descriptors are passed as a plain dict of int32 numpy arrays (struct of arrays):

    prefix_len, n_branches, branch_begin, page_begin, n_pages, tail_off, tail_len   [n_req]
    br_kv_off, br_kv_len, br_q_len                                                  [n_br]
    page_ids                                                                        [sum n_pages]
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aspd_oracle.c")
_LIB = os.path.join(_HERE, "libaspd_oracle.so")

MODE_BRANCH = 0
MODE_SERIAL = 1
MASK_BRANCH_INVISIBLE = 0   # Eq. 2-3
MASK_SHARED = 1             # the visible mask of the attention-mask ablation

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.aspd_oracle_rope.restype = None
        for name in ("aspd_oracle_dense_positions", "aspd_oracle_dense_visible", "aspd_oracle_dense_attn",
                     "aspd_oracle_new_tokens", "aspd_oracle_kv_append", "aspd_oracle_attn", "aspd_oracle_attn_at",
                     "aspd_oracle_visible_slots", "aspd_oracle_threads", "aspd_oracle_dense_visible_shared",
                     "aspd_oracle_dense_attn_shared", "aspd_oracle_attn_masked", "aspd_oracle_visible_slots_masked"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(lib().aspd_oracle_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def rope(x, pos: float, theta: float) -> np.ndarray:
    x = _f64(x)
    out = np.empty_like(x)
    lib().aspd_oracle_rope(_p(x), ctypes.c_int(x.shape[-1]), ctypes.c_double(pos), ctypes.c_double(theta), _p(out))
    return out


# ----------------------------------------------------------------------------- dense form
def dense_positions(branch, stage) -> np.ndarray:
    branch, stage = _i32(branch), _i32(stage)
    pos = np.empty(len(branch), dtype=np.int32)
    rc = lib().aspd_oracle_dense_positions(len(branch), _p(branch), _p(stage), _p(pos))
    assert rc == 0
    return pos


def dense_visible(branch, stage, pos=None) -> np.ndarray:
    branch, stage = _i32(branch), _i32(stage)
    pos = dense_positions(branch, stage) if pos is None else _i32(pos)
    L = len(branch)
    vis = np.zeros((L, L), dtype=np.uint8)
    rc = lib().aspd_oracle_dense_visible(L, _p(branch), _p(stage), _p(pos), _p(vis))
    assert rc == 0
    return vis


def dense_visible_shared(pos) -> np.ndarray:
    """Visible ("Shared") mask of the ablation: i sees j iff pos[j] < pos[i], or j == i."""
    pos = _i32(pos)
    L = len(pos)
    vis = np.zeros((L, L), dtype=np.uint8)
    rc = lib().aspd_oracle_dense_visible_shared(L, _p(pos), _p(vis))
    assert rc == 0
    return vis


def dense_attn(q, k, v, branch, stage, theta: float, sm_scale: float, mask: int = MASK_BRANCH_INVISIBLE) -> np.ndarray:
    """q [L][Hq][d], k/v [L][Hkv][d] raw (un-rotated); returns out [L][Hq][d]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    branch, stage = _i32(branch), _i32(stage)
    L, Hq, d = q.shape
    Hkv = k.shape[1]
    out = np.empty_like(q)
    fn = lib().aspd_oracle_dense_attn_shared if mask == MASK_SHARED else lib().aspd_oracle_dense_attn
    rc = fn(L, Hq, Hkv, d, ctypes.c_double(theta), ctypes.c_double(sm_scale),
            _p(q), _p(k), _p(v), _p(branch), _p(stage), _p(out))
    assert rc == 0, rc
    return out


# ------------------------------------------------------------------------ descriptor form
_REQ_KEYS = ("prefix_len", "n_branches", "branch_begin", "page_begin", "n_pages", "tail_off", "tail_len")
_BR_KEYS = ("br_kv_off", "br_kv_len", "br_q_len")


def _desc(desc):
    d = {k: _i32(desc[k]) for k in _REQ_KEYS + _BR_KEYS + ("page_ids",)}
    return d


def n_new_tokens(desc, mode: int) -> int:
    d = _desc(desc)
    if mode == MODE_SERIAL:
        return len(d["prefix_len"])
    n = 0
    for r in range(len(d["prefix_len"])):
        b0 = int(d["branch_begin"][r])
        n += int(np.clip(d["br_q_len"][b0:b0 + int(d["n_branches"][r])], 0, None).sum())
    return n


def new_tokens(desc, mode: int):
    """Position ID (Eq. 4), logical slot and request of every new token."""
    d = _desc(desc)
    n = n_new_tokens(d, mode)
    pos = np.empty(n, dtype=np.int32)
    slot = np.empty(n, dtype=np.int32)
    req = np.empty(n, dtype=np.int32)
    rc = lib().aspd_oracle_new_tokens(len(d["prefix_len"]), mode, _p(d["prefix_len"]), _p(d["n_branches"]),
                                      _p(d["branch_begin"]), _p(d["tail_off"]), _p(d["tail_len"]),
                                      _p(d["br_kv_off"]), _p(d["br_kv_len"]), _p(d["br_q_len"]),
                                      _p(pos), _p(slot), _p(req))
    assert rc == n, (rc, n)
    return pos, slot, req


def make_pools(n_pool_pages: int, Hkv: int, page_size: int, d: int):
    shape = (n_pool_pages, Hkv, page_size, d)
    return np.zeros(shape, dtype=np.float64), np.zeros(shape, dtype=np.float64)


def kv_append(desc, k_new, v_new, pos, req, slot, k_pool, v_pool, theta: float) -> None:
    """a3: RoPE the new keys at ``pos`` and scatter K', V into the paged fp64 pools (in place)."""
    d = _desc(desc)
    k_new, v_new = _f64(k_new), _f64(v_new)
    pos, req, slot = _i32(pos), _i32(req), _i32(slot)
    n_new, Hkv, hd = k_new.shape
    assert k_pool.dtype == np.float64 and k_pool.flags.c_contiguous and v_pool.flags.c_contiguous
    page_size = k_pool.shape[2]
    rc = lib().aspd_oracle_kv_append(n_new, Hkv, hd, page_size, ctypes.c_double(theta), _p(k_new), _p(v_new),
                                     _p(pos), _p(req), _p(slot), _p(d["page_begin"]), _p(d["page_ids"]),
                                     _p(k_pool), _p(v_pool))
    assert rc == 0


def attn(desc, mode: int, q, k_pool, v_pool, theta: float, sm_scale: float, q_pos=None,
         mask: int = MASK_BRANCH_INVISIBLE) -> np.ndarray:
    """a4-a7 (mode 0) / a9 (mode 1): out [n_new][Hq][d] for raw queries q [n_new][Hq][d].
    ``q_pos``: query positions of a position-ID variant (default: Eq. 4); ``mask``: the
    branch-invisible mask of Eq. 2-3 or the ablation's visible one."""
    d = _desc(desc)
    q = _f64(q)
    n_new, Hq, hd = q.shape
    assert n_new == n_new_tokens(d, mode)
    Hkv, page_size = k_pool.shape[1], k_pool.shape[2]
    out = np.empty_like(q)
    if mask != MASK_BRANCH_INVISIBLE:
        qp = None if q_pos is None else _i32(q_pos)
        rc = lib().aspd_oracle_attn_masked(len(d["prefix_len"]), mode, Hq, Hkv, hd, page_size, ctypes.c_double(theta),
                                           ctypes.c_double(sm_scale), _p(d["prefix_len"]), _p(d["n_branches"]),
                                           _p(d["branch_begin"]), _p(d["page_begin"]), _p(d["tail_off"]), _p(d["tail_len"]),
                                           _p(d["br_kv_off"]), _p(d["br_kv_len"]), _p(d["br_q_len"]), _p(d["page_ids"]),
                                           _p(q), None if qp is None else _p(qp), ctypes.c_int(mask), _p(k_pool), _p(v_pool), _p(out))
        assert rc == 0, rc
        return out
    if q_pos is not None:
        qp = _i32(q_pos)
        assert len(qp) == n_new
        rc = lib().aspd_oracle_attn_at(len(d["prefix_len"]), mode, Hq, Hkv, hd, page_size, ctypes.c_double(theta),
                                       ctypes.c_double(sm_scale), _p(d["prefix_len"]), _p(d["n_branches"]),
                                       _p(d["branch_begin"]), _p(d["page_begin"]), _p(d["tail_off"]), _p(d["tail_len"]),
                                       _p(d["br_kv_off"]), _p(d["br_kv_len"]), _p(d["br_q_len"]), _p(d["page_ids"]),
                                       _p(q), _p(qp), _p(k_pool), _p(v_pool), _p(out))
        assert rc == 0, rc
        return out
    rc = lib().aspd_oracle_attn(len(d["prefix_len"]), mode, Hq, Hkv, hd, page_size, ctypes.c_double(theta),
                                ctypes.c_double(sm_scale), _p(d["prefix_len"]), _p(d["n_branches"]),
                                _p(d["branch_begin"]), _p(d["page_begin"]), _p(d["tail_off"]), _p(d["tail_len"]),
                                _p(d["br_kv_off"]), _p(d["br_kv_len"]), _p(d["br_q_len"]), _p(d["page_ids"]),
                                _p(q), _p(k_pool), _p(v_pool), _p(out))
    assert rc == 0, rc
    return out


def visible_slots(desc, mode: int, n_slots: int, mask: int = MASK_BRANCH_INVISIBLE) -> np.ndarray:
    """[n_new][n_slots] 0/1: logical slots of its own request that each new token may see."""
    d = _desc(desc)
    n = n_new_tokens(d, mode)
    vis = np.zeros((n, n_slots), dtype=np.uint8)
    rc = lib().aspd_oracle_visible_slots_masked(len(d["prefix_len"]), mode, n_slots, _p(d["prefix_len"]),
                                                _p(d["n_branches"]), _p(d["branch_begin"]), _p(d["tail_off"]),
                                                _p(d["tail_len"]), _p(d["br_kv_off"]), _p(d["br_kv_len"]),
                                                _p(d["br_q_len"]), ctypes.c_int(mask), _p(vis))
    assert rc == n
    return vis
