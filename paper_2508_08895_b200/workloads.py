"""Seeded synthetic workloads shaped like the paper's decoding traffic.

This module is the one piece shared by the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds no arithmetic of the method: no position IDs, no RoPE, no mask, no
softmax.  It only draws raw Q/K/V values from a counter-based generator, rounds them once to
the storage dtype, lays out logical slots (shared prefix, page-aligned branch regions, tail)
and assigns physical pages by a seeded permutation.  Both sides derive positions, slots of
new tokens and visible sets from the descriptors with their own code.

The shapes follow the paper's parallel segments: 2-8 branches (average branch numbers of
2.4-3.2 in its Tables 2 and 5), branches of tens to a few hundred tokens (its Fix-32 remark in
the position-ID ablation), shared contexts of 1k-16k tokens (8k/12k training contexts,
retrieval-augmented prompts).  The datasets themselves are not used.

A workload is a list of phases.  Each phase is one call sequence ``kv_append -> attention``
(attention skipped for pure cache-fill phases) described by a descriptor dict
(struct of int32 arrays, see ``DESC_REQ_KEYS`` / ``DESC_BR_KEYS``) plus raw ``k_new``,
``v_new`` and ``q`` for that phase's new tokens.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

MODE_BRANCH = 0
MODE_SERIAL = 1

DESC_REQ_KEYS = ("prefix_len", "n_branches", "branch_begin", "page_begin", "n_pages", "tail_off", "tail_len")
DESC_BR_KEYS = ("br_kv_off", "br_kv_len", "br_q_len")

SEED_BASE = 0xA5BD0000

# --------------------------------------------------------------------- counter-based RNG
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 counters (vectorised, wraps modulo 2^64)."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def uniform_u64(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """count 64-bit words; word i depends only on (seed, stream, start + i)."""
    with np.errstate(over="ignore"):
        base = _splitmix64(np.array([(seed * 0x100000001B3 + stream) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0]
        ctr = np.arange(start, start + count, dtype=np.uint64)
        return _splitmix64(ctr ^ base)


def normal(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """count standard normals (fp64); element i depends only on (seed, stream, start + i)."""
    with np.errstate(over="ignore"):
        a = uniform_u64(seed, stream, 2 * start, 2 * count)
    u1 = ((a[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)  # (0, 1]
    u2 = (a[1::2] >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)          # [0, 1)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def randint(seed: int, stream: int, index: int, lo: int, hi: int) -> int:
    """Uniform integer in [lo, hi] from one counter."""
    w = int(uniform_u64(seed, stream, index, 1)[0])
    return lo + w % (hi - lo + 1)


def permutation(seed: int, stream: int, n: int) -> np.ndarray:
    keys = uniform_u64(seed, stream, 0, n)
    return np.argsort(keys, kind="stable").astype(np.int32)


# ------------------------------------------------------------------ storage-dtype rounding
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to the nearest bf16 (ties to even); returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32)


def bf16_bits(x32: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    return (np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


# --------------------------------------------------------------------------- containers
@dataclass
class Phase:
    mode: int                       # MODE_BRANCH / MODE_SERIAL
    desc: Dict[str, np.ndarray]     # descriptors AFTER this phase's append
    k_new: np.ndarray               # [n_new][Hkv][d] float32 (storage-rounded)
    v_new: np.ndarray
    q: Optional[np.ndarray]         # [n_new][Hq][d] or None for a pure cache fill
    compare: bool = False           # attention output of this phase is checked / timed
    label: str = ""


@dataclass
class Workload:
    name: str
    Hq: int
    Hkv: int
    d: int
    page_size: int
    dtype: str                      # "bf16" | "f32"
    theta: float
    sm_scale: float
    n_pool_pages: int
    phases: List[Phase] = field(default_factory=list)
    seed: int = 0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


def _ceil_div(a: int, b: int) -> int:
    return -(-a // b)


# --------------------------------------------------------------------- layout + phases
class _Request:
    """Logical-slot layout of one request: prefix, page-aligned branch regions, tail."""

    def __init__(self, P: int, branch_caps: List[int], tail_cap: int, page: int):
        self.P = P
        off = _ceil_div(P, page) * page
        self.br_off = []
        for cap in branch_caps:
            self.br_off.append(off)
            off += _ceil_div(max(cap, 1), page) * page
        self.tail_off = off
        off += _ceil_div(max(tail_cap, 0), page) * page
        self.n_slots = off
        self.n_pages = _ceil_div(off, page)


def _make_desc(reqs, page_tables, br_len, br_q, tail_len, with_branches=True):
    """Assemble the struct-of-arrays descriptor for all requests."""
    d = {k: [] for k in DESC_REQ_KEYS + DESC_BR_KEYS}
    pages = []
    for r, rq in enumerate(reqs):
        d["prefix_len"].append(rq.P)
        nb = len(rq.br_off) if with_branches else 0
        d["n_branches"].append(nb)
        d["branch_begin"].append(len(d["br_kv_off"]))
        d["page_begin"].append(len(pages))
        d["n_pages"].append(rq.n_pages)
        d["tail_off"].append(rq.tail_off)
        d["tail_len"].append(tail_len[r])
        for b in range(nb):
            d["br_kv_off"].append(rq.br_off[b])
            d["br_kv_len"].append(br_len[r][b])
            d["br_q_len"].append(br_q[r][b])
        pages.extend(page_tables[r].tolist())
    out = {k: np.asarray(v, dtype=np.int32) for k, v in d.items()}
    out["page_ids"] = np.asarray(pages, dtype=np.int32)
    return out


class _Values:
    """Raw K/V/Q of (request, logical slot): a pure function of (seed, request, slot)."""

    def __init__(self, seed, Hq, Hkv, d, dtype, max_slots):
        self.seed, self.Hq, self.Hkv, self.d, self.dtype, self.max_slots = seed, Hq, Hkv, d, dtype, max_slots

    def _draw(self, stream, r, slots, width):
        slots = np.asarray(slots, dtype=np.int64)
        out = np.empty((len(slots), width), dtype=np.float32)
        # contiguous runs are generated in one call
        i = 0
        while i < len(slots):
            j = i
            while j + 1 < len(slots) and slots[j + 1] == slots[j] + 1:
                j += 1
            start = (r * self.max_slots + int(slots[i])) * width
            vals = normal(self.seed, stream, start, (j - i + 1) * width)
            out[i:j + 1] = round_storage(vals, self.dtype).reshape(j - i + 1, width)
            i = j + 1
        return out

    def k(self, r, slots):
        return self._draw(1, r, slots, self.Hkv * self.d).reshape(-1, self.Hkv, self.d)

    def v(self, r, slots):
        return self._draw(2, r, slots, self.Hkv * self.d).reshape(-1, self.Hkv, self.d)

    def q(self, r, slots):
        return self._draw(3, r, slots, self.Hq * self.d).reshape(-1, self.Hq, self.d)


def _phase(vals, mode, desc, slots_per_req, want_q, compare, label):
    ks, vs, qs = [], [], []
    for r, slots in enumerate(slots_per_req):
        if len(slots) == 0:
            continue
        ks.append(vals.k(r, slots))
        vs.append(vals.v(r, slots))
        if want_q:
            qs.append(vals.q(r, slots))
    Hkv, Hq, d = vals.Hkv, vals.Hq, vals.d
    k_new = np.concatenate(ks) if ks else np.zeros((0, Hkv, d), np.float32)
    v_new = np.concatenate(vs) if vs else np.zeros((0, Hkv, d), np.float32)
    q = (np.concatenate(qs) if qs else np.zeros((0, Hq, d), np.float32)) if want_q else None
    return Phase(mode=mode, desc=desc, k_new=k_new, v_new=v_new, q=q, compare=compare, label=label)


def build_segment_workload(name: str, seed: int, Hq: int, Hkv: int, d: int, dtype: str, theta: float,
                           prefix_lens: List[int], prior_lens: List[List[int]], q_lens: List[List[int]],
                           serial_steps: int = 0, page_size: int = 16, sm_scale: Optional[float] = None,
                           extra_pool_pages: int = 3, serial_without_branches: bool = False) -> Workload:
    """General builder.

    Per request r: a shared prefix of ``prefix_lens[r]`` tokens; branch b holds
    ``prior_lens[r][b]`` tokens before the measured step and receives ``q_lens[r][b]`` new
    query tokens in it (0 = a branch that already finished).  Then ``serial_steps`` serial
    decode steps run over the merged cache.

    Phases: (1) prefix fill, expressed as a branch-mode call with an empty prefix and one
    "branch" that is the prefix itself; (2) prior branch tokens; (3) the measured parallel
    step; (4..) serial steps.  Every phase's new tokens are ordered request-major, then
    branch, then token.
    """
    n_req = len(prefix_lens)
    sm_scale = float(sm_scale if sm_scale is not None else 1.0 / np.sqrt(d))
    reqs = []
    for r in range(n_req):
        caps = [prior_lens[r][b] + q_lens[r][b] for b in range(len(prior_lens[r]))]
        reqs.append(_Request(prefix_lens[r], caps, serial_steps, page_size))
    total_pages = sum(rq.n_pages for rq in reqs)
    n_pool_pages = total_pages + extra_pool_pages
    perm = permutation(seed, 7, n_pool_pages)
    page_tables, at = [], 0
    for rq in reqs:
        page_tables.append(perm[at:at + rq.n_pages])
        at += rq.n_pages
    vals = _Values(seed, Hq, Hkv, d, dtype, max(rq.n_slots for rq in reqs) + 1)
    wl = Workload(name=name, Hq=Hq, Hkv=Hkv, d=d, page_size=page_size, dtype=dtype, theta=float(theta),
                  sm_scale=sm_scale, n_pool_pages=n_pool_pages, seed=seed)
    zeros_tail = [0] * n_req

    # (1) prefix fill: P = 0, one branch [0, P) with q_len = P
    pre_reqs = []
    for rq in reqs:
        p = _Request(0, [rq.P], 0, page_size)
        p.n_pages, p.n_slots, p.tail_off = rq.n_pages, rq.n_slots, rq.tail_off
        pre_reqs.append(p)
    if any(rq.P > 0 for rq in reqs):
        desc = _make_desc(pre_reqs, page_tables, [[rq.P] for rq in reqs], [[rq.P] for rq in reqs], zeros_tail)
        wl.phases.append(_phase(vals, MODE_BRANCH, desc, [np.arange(rq.P) for rq in reqs], False, False, "fill-prefix"))

    # (2) prior branch tokens
    if any(sum(p) > 0 for p in prior_lens):
        desc = _make_desc(reqs, page_tables, prior_lens, prior_lens, zeros_tail)
        slots = [np.concatenate([np.arange(rq.br_off[b], rq.br_off[b] + prior_lens[r][b]) for b in range(len(rq.br_off))]
                                + [np.zeros(0, np.int64)]).astype(np.int64) for r, rq in enumerate(reqs)]
        wl.phases.append(_phase(vals, MODE_BRANCH, desc, slots, False, False, "fill-branches"))

    # (3) the measured parallel step
    final_len = [[prior_lens[r][b] + q_lens[r][b] for b in range(len(prior_lens[r]))] for r in range(n_req)]
    if any(sum(ql) > 0 for ql in q_lens):
        desc = _make_desc(reqs, page_tables, final_len, q_lens, zeros_tail)
        slots = [np.concatenate([np.arange(rq.br_off[b] + prior_lens[r][b], rq.br_off[b] + final_len[r][b])
                                 for b in range(len(rq.br_off))] + [np.zeros(0, np.int64)]).astype(np.int64)
                 for r, rq in enumerate(reqs)]
        wl.phases.append(_phase(vals, MODE_BRANCH, desc, slots, True, True, "parallel-step"))

    # (4) serial steps over the merged cache (the merge itself moves nothing)
    for s in range(serial_steps):
        zero_q = [[0] * len(p) for p in prior_lens]
        desc = _make_desc(reqs, page_tables, final_len, zero_q, [s + 1] * n_req, with_branches=not serial_without_branches)
        slots = [np.array([rq.tail_off + s], dtype=np.int64) for rq in reqs]
        wl.phases.append(_phase(vals, MODE_SERIAL, desc, slots, True, True, f"serial-{s}"))
    return wl


def build_two_stage_workload(name: str, seed: int, Hq: int, Hkv: int, d: int, dtype: str, theta: float, prefix: int,
                             stage1: List[int], tail1: int, prior2: List[int], q2: List[int], serial_steps: int = 1,
                             page_size: int = 16) -> Workload:
    """One request that has already been through a parallel stage and opens a second one (the
    engine switches between serial and parallel decoding repeatedly).

    Cache before the measured step: ``prefix`` tokens, the merged branches of the first stage
    (``stage1`` lengths), ``tail1`` serial tokens decoded after it, and ``prior2`` tokens in each
    branch of the second stage.  The measured step adds ``q2`` tokens per second-stage branch;
    then ``serial_steps`` serial steps follow.  Regions of the earlier stage are marked with
    ``br_q_len = -1`` (visible to every branch of the current stage).
    """
    n1, n2 = len(stage1), len(prior2)
    caps = list(stage1) + [tail1] + [prior2[b] + q2[b] for b in range(n2)]
    rq = _Request(prefix, caps, serial_steps, page_size)
    n_pool_pages = rq.n_pages + 3
    table = permutation(seed, 7, n_pool_pages)[: rq.n_pages]
    vals = _Values(seed, Hq, Hkv, d, dtype, rq.n_slots + 1)
    wl = Workload(name=name, Hq=Hq, Hkv=Hkv, d=d, page_size=page_size, dtype=dtype, theta=float(theta),
                  sm_scale=float(1.0 / np.sqrt(d)), n_pool_pages=n_pool_pages, seed=seed)

    def desc(P, regions, tail_off, tail_len):
        """regions: list of (slot offset, kv_len, q_len)."""
        out = {"prefix_len": [P], "n_branches": [len(regions)], "branch_begin": [0], "page_begin": [0],
               "n_pages": [rq.n_pages], "tail_off": [tail_off], "tail_len": [tail_len],
               "br_kv_off": [r[0] for r in regions], "br_kv_len": [r[1] for r in regions], "br_q_len": [r[2] for r in regions]}
        out = {k: np.asarray(v, dtype=np.int32) for k, v in out.items()}
        out["page_ids"] = np.asarray(table, dtype=np.int32)
        return out

    def span(off, lo, hi):
        return np.arange(off + lo, off + hi, dtype=np.int64)

    off1, off_t1, off2 = rq.br_off[:n1], rq.br_off[n1], rq.br_off[n1 + 1:]
    # prefix (an empty prefix plus one "branch" that is the prefix itself), then the first stage
    wl.phases.append(_phase(vals, MODE_BRANCH, desc(0, [(0, prefix, prefix)], rq.tail_off, 0), [span(0, 0, prefix)],
                            False, False, "fill-prefix"))
    wl.phases.append(_phase(vals, MODE_BRANCH, desc(prefix, [(off1[b], stage1[b], stage1[b]) for b in range(n1)], rq.tail_off, 0),
                            [np.concatenate([span(off1[b], 0, stage1[b]) for b in range(n1)])], False, False, "fill-stage1"))
    # serial tokens between the stages, one step each
    merged1 = [(off1[b], stage1[b], 0) for b in range(n1)]
    for s_ in range(tail1):
        wl.phases.append(_phase(vals, MODE_SERIAL, desc(prefix, merged1, off_t1, s_ + 1), [span(off_t1, s_, s_ + 1)],
                                False, False, f"fill-tail1-{s_}"))
    shared = [(off1[b], stage1[b], -1) for b in range(n1)] + ([(off_t1, tail1, -1)] if tail1 > 0 else [])
    if sum(prior2) > 0:
        wl.phases.append(_phase(vals, MODE_BRANCH, desc(prefix, shared + [(off2[b], prior2[b], prior2[b]) for b in range(n2)],
                                                        rq.tail_off, 0),
                                [np.concatenate([span(off2[b], 0, prior2[b]) for b in range(n2)])], False, False, "fill-stage2"))
    final2 = [prior2[b] + q2[b] for b in range(n2)]
    wl.phases.append(_phase(vals, MODE_BRANCH, desc(prefix, shared + [(off2[b], final2[b], q2[b]) for b in range(n2)], rq.tail_off, 0),
                            [np.concatenate([span(off2[b], prior2[b], final2[b]) for b in range(n2)])], True, True, "parallel-step"))
    for s_ in range(serial_steps):
        wl.phases.append(_phase(vals, MODE_SERIAL, desc(prefix, shared + [(off2[b], final2[b], 0) for b in range(n2)],
                                                        rq.tail_off, s_ + 1),
                                [span(rq.tail_off, s_, s_ + 1)], True, True, f"serial-{s_}"))
    return wl


# ------------------------------------------------------------------- the five configurations
def config_tiny(seed: int = SEED_BASE + 0) -> Workload:
    """4 q heads, 1 KV head, d 64, fp32; prefix 256; branches hold 16/9/23 + 1 new; theta 1e4."""
    return build_segment_workload("tiny-f32", seed, 4, 1, 64, "f32", 10000.0, [256], [[16, 9, 23]], [[1, 1, 1]])


def config_qwen7b_layer(seed: int = SEED_BASE + 1, theta: float = 1.0e6) -> Workload:
    """28/4 heads, d 128, bf16; prefix 2048; 4 branches of 128 tokens + 1 new each."""
    return build_segment_workload("qwen7b-layer", seed, 28, 4, 128, "bf16", theta, [2048], [[128] * 4], [[1] * 4])


def config_branch_open(seed: int = SEED_BASE + 2, theta: float = 1.0e6, serial_steps: int = 64) -> Workload:
    """Prefix 1024; 6 branches open with 12-token headers (72 queries); merge; 64 serial steps."""
    return build_segment_workload("branch-open", seed, 28, 4, 128, "bf16", theta, [1024], [[0] * 6], [[12] * 6],
                                  serial_steps=serial_steps)


def config_long_rag(seed: int = SEED_BASE + 3, theta: float = 1.0e6, prefix: int = 16384) -> Workload:
    """Prefix 16384; 8 branches of uniform 32-256 prior tokens + 1 new each."""
    prior = [randint(seed, 11, b, 32, 256) for b in range(8)]
    return build_segment_workload("long-rag", seed, 28, 4, 128, "bf16", theta, [prefix], [prior], [[1] * 8])


def serving_mix_lengths(seed: int = SEED_BASE + 4, n_req: int = 32):
    """Lengths of the batched serving mix: prefix log-uniform 512-8192, 1-8 branches, 1-256 prior tokens."""
    prefix, prior = [], []
    for r in range(n_req):
        u = (int(uniform_u64(seed, 12, r, 1)[0]) >> 11) / 9007199254740992.0
        prefix.append(int(round(512.0 * (8192.0 / 512.0) ** u)))
        nb = randint(seed, 13, r, 1, 8)
        prior.append([randint(seed, 14, r * 8 + b, 1, 256) for b in range(nb)])
    return prefix, prior


def config_serving_mix(seed: int = SEED_BASE + 4, theta: float = 1.0e6, n_req: int = 32) -> Workload:
    """32 requests, ragged: prefix log-uniform 512-8192, 1-8 branches, branch length 1-256, +1 new each."""
    prefix, prior = serving_mix_lengths(seed, n_req)
    return build_segment_workload("serving-mix", seed, 28, 4, 128, "bf16", theta, prefix, prior,
                                  [[1] * len(p) for p in prior])


def config_masked_prefill(seed: int = SEED_BASE + 5, theta: float = 1.0e6, n_req: int = 32) -> Workload:
    """The serving mix's requests in the teacher-forcing layout: every branch's tokens (its 1-256
    earlier ones and the new one) are query tokens of ONE step over the request's cached prefix."""
    prefix, prior = serving_mix_lengths(seed, n_req)
    return build_segment_workload("masked-prefill", seed, 28, 4, 128, "bf16", theta, prefix, [[0] * len(p) for p in prior],
                                  [[x + 1 for x in p] for p in prior])


def config_serving_mix_serial(seed: int = SEED_BASE + 4, theta: float = 1.0e6, n_req: int = 32) -> Workload:
    """The serving mix one step later: the segment has ended, every request decodes one serial
    token over its merged cache (prefix, all branches, tail) -- nothing was moved or recomputed."""
    prefix, prior = serving_mix_lengths(seed, n_req)
    return build_segment_workload("serving-mix-serial", seed, 28, 4, 128, "bf16", theta, prefix, prior,
                                  [[1] * len(p) for p in prior], serial_steps=1)


CONFIGS = {
    "tiny-f32": config_tiny,
    "qwen7b-layer": config_qwen7b_layer,
    "branch-open": config_branch_open,
    "long-rag": config_long_rag,
    "serving-mix": config_serving_mix,
    "masked-prefill": config_masked_prefill,
    "serving-mix-serial": config_serving_mix_serial,
}
