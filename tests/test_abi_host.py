"""CPU-only checks of the C ABI: the library loads, exports what the header declares, and its
host-side integer logic (positions, slots, mask membership, validation, work list) is exact."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2508_08895_b200 import binding as B, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "aspd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aspd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = B.lib()
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(L, name), name
    assert set(B.EXPORTS) == set(names)


def test_struct_sizes_and_strerror():
    assert B.REQUEST_DTYPE.itemsize == 28 and B.BRANCH_DTYPE.itemsize == 16 and B.ITEM_DTYPE.itemsize == 40
    assert ctypes.sizeof(B.Shape) == 28
    assert ctypes.sizeof(B.Tuning) == 40 and ctypes.sizeof(B.PlanInfo) == 80      # 10 and 14 int32 + 3 int64, as in aspd.h
    # the header itself, through a C compiler: the binding's structs have the sizes C gives them
    import subprocess, tempfile
    src = ('#include <stdio.h>\n#include "aspd.h"\nint main(void) { printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(aspd_request_t), '
           'sizeof(aspd_branch_t), sizeof(aspd_shape_t), sizeof(aspd_tuning_t), sizeof(aspd_item_t), sizeof(aspd_plan_info_t)); return 0; }\n')
    with tempfile.TemporaryDirectory() as tmp:
        open(os.path.join(tmp, "s.c"), "w").write(src)
        subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), os.path.join(tmp, "s.c"), "-o", os.path.join(tmp, "s")],
                       check=True)
        sizes = [int(x) for x in subprocess.run([os.path.join(tmp, "s")], capture_output=True, text=True, check=True).stdout.split()]
    assert sizes == [B.REQUEST_DTYPE.itemsize, B.BRANCH_DTYPE.itemsize, ctypes.sizeof(B.Shape), ctypes.sizeof(B.Tuning),
                     B.ITEM_DTYPE.itemsize, ctypes.sizeof(B.PlanInfo)]
    assert B.strerror(0) == "ok"
    for code in range(-7, 0):
        assert B.strerror(code) not in ("ok", "unknown status")


def small_workloads():
    yield W.build_segment_workload("a", 3, 4, 2, 64, "f32", 1e4, [5], [[2, 1, 2]], [[1, 0, 1]], serial_steps=2)
    yield W.build_segment_workload("b", 4, 28, 4, 128, "bf16", 1e6, [15, 16, 17, 0], [[16, 1], [17], [0, 0, 33], [4]],
                                   [[1, 1], [1], [12, 5, 1], [1]], serial_steps=1)
    yield W.config_tiny()
    yield W.build_two_stage_workload("ts", 5, 28, 4, 128, "bf16", 1e6, 37, [30, 1, 17], 3, [5, 0, 40], [1, 2, 1], serial_steps=2)
    yield W.config_branch_open(serial_steps=3)


def test_positions_and_slots_match_oracle_bit_exact():
    for wl in small_workloads():
        for ph in wl.phases:
            pos, slot, req = B.positions(ph.desc, ph.mode)
            opos, oslot, oreq = oracle.new_tokens(ph.desc, ph.mode)
            np.testing.assert_array_equal(pos, opos)
            np.testing.assert_array_equal(slot, oslot)
            np.testing.assert_array_equal(req, oreq)
            assert B.count_new_tokens(ph.desc, ph.mode) == len(opos)


def test_positions_closed_forms():
    # parallel token k of a branch: P + k for every branch; serial: P + sum(len) + tail - 1
    wl = W.build_segment_workload("c", 5, 4, 2, 64, "f32", 1e4, [40], [[3, 0, 7]], [[1, 1, 1]], serial_steps=2)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    pos, slot, _ = B.positions(par.desc, B.MODE_BRANCH)
    assert pos.tolist() == [43, 40, 47]
    assert slot.tolist() == [48 + 3, 64 + 0, 80 + 7]
    ser = [p for p in wl.phases if p.label == "serial-1"][0]
    pos, slot, _ = B.positions(ser.desc, B.MODE_SERIAL)
    assert pos.tolist() == [40 + 4 + 1 + 8 + 1]
    assert slot.tolist() == [96 + 1]


def test_stage_start_is_derived_behind_the_c_abi():
    """Eq. 4's stage_start without any help from the Python binding: the raw C structs are filled
    with numpy (pos_start = ASPD_POS_AUTO) and handed to aspd_positions through ctypes; the result
    is the oracle's, bit for bit, for a first stage (prefix only) and a second stage (prefix + the
    merged branches of the first + the serial tokens between them).  A caller-given pos_start >= 0
    is taken as it is."""
    import ctypes
    L = B.lib()
    one = W.build_segment_workload("s1", 11, 4, 2, 64, "f32", 1e4, [37, 5], [[3, 0, 7], [2]], [[1, 2, 1], [4]])
    two = W.build_two_stage_workload("s2", 12, 4, 2, 64, "f32", 1e4, 9, [3, 1, 2], 2, [4, 0, 6], [1, 2, 1])
    for wl, want_start in ((one, [37, 37, 37, 5]), (two, None)):
        d = [p for p in wl.phases if p.label == "parallel-step"][0].desc
        n_req, n_br = len(d["prefix_len"]), len(d["br_kv_off"])
        req = np.zeros(n_req, dtype=np.dtype([(n, np.int32) for n in ("prefix_len", "n_branches", "branch_begin", "page_begin",
                                                                       "n_pages", "tail_off", "tail_len")]))
        for name in req.dtype.names:
            req[name] = d[name]
        br = np.zeros(n_br, dtype=np.dtype([(n, np.int32) for n in ("kv_off", "kv_len", "pos_start", "q_len")]))
        br["kv_off"], br["kv_len"], br["q_len"], br["pos_start"] = d["br_kv_off"], d["br_kv_len"], d["br_q_len"], -1
        assert req.itemsize == 28 and br.itemsize == 16
        n = L.aspd_count_new_tokens(req.ctypes.data, br.ctypes.data, n_req, 0)
        opos, oslot, oreq = oracle.new_tokens(d, oracle.MODE_BRANCH)
        assert n == len(opos) > 0
        pos, slot, rq = (np.full(n, -7, np.int32) for _ in range(3))
        assert L.aspd_positions(req.ctypes.data, br.ctypes.data, n_req, 0, pos.ctypes.data, slot.ctypes.data, rq.ctypes.data) == 0
        np.testing.assert_array_equal(pos, opos)
        np.testing.assert_array_equal(slot, oslot)
        np.testing.assert_array_equal(rq, oreq)
        if want_start is not None:      # closed form: P + k
            k = np.concatenate([np.arange(l - q, l) for l, q in zip(d["br_kv_len"], d["br_q_len"]) if q > 0])
            first = np.concatenate([[s_] * q for s_, q in zip(want_start, d["br_q_len"]) if q > 0])
            np.testing.assert_array_equal(pos, first + k)
        else:                           # second stage: 9 prefix + (3 + 1 + 2) merged + 2 serial tokens = 17
            live = d["br_q_len"] > 0
            k = np.concatenate([np.arange(l - q, l) for l, q in zip(d["br_kv_len"][live], d["br_q_len"][live])])
            np.testing.assert_array_equal(pos, 17 + k)
        # a caller-given start (a position-ID variant) is used as given
        br["pos_start"] = 1000
        assert L.aspd_positions(req.ctypes.data, br.ctypes.data, n_req, 0, pos.ctypes.data, slot.ctypes.data, rq.ctypes.data) == 0
        live = d["br_q_len"] > 0
        k = np.concatenate([np.arange(l - q, l) for l, q in zip(d["br_kv_len"][live], d["br_q_len"][live])])
        np.testing.assert_array_equal(pos, 1000 + k)
        br["pos_start"] = -2
        assert L.aspd_positions(req.ctypes.data, br.ctypes.data, n_req, 0, pos.ctypes.data, slot.ctypes.data, rq.ctypes.data) == -2


def test_visible_slots_match_oracle_bit_exact():
    for wl in small_workloads():
        for ph in wl.phases:
            n_slots = int(ph.desc["n_pages"].max()) * wl.page_size
            np.testing.assert_array_equal(B.visible_slots(ph.desc, ph.mode, n_slots),
                                          oracle.visible_slots(ph.desc, ph.mode, n_slots))


def _shape(wl):
    return B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)


def _check_cover(wl, ph, plan, chunk=0, dealt=False, mask=0):
    """The plan's work items, expanded through its stream-page list and the per-token visible
    ranges to (token, KV head, logical slot) triples, are exactly the oracle's visible sets."""
    dealt = dealt or bool(plan.info.dealt)
    n_slots = int(ph.desc["n_pages"].max()) * wl.page_size
    vis = oracle.visible_slots(ph.desc, ph.mode, n_slots, mask=mask)
    _, _, treq = oracle.new_tokens(ph.desc, ph.mode)
    page_ids, n_valid = plan.stream_pages()
    pe, lo, hi = plan.token_ranges()
    shared = bool(mask) and ph.mode == B.MODE_BRANCH
    below, page_in_branch = plan.shared_mask_tables() if shared else (np.zeros(plan.n_new, np.int32), None)
    # physical page -> (request, logical page)
    where = {}
    for r in range(len(ph.desc["prefix_len"])):
        pb = int(ph.desc["page_begin"][r])
        for lp in range(int(ph.desc["n_pages"][r])):
            where[int(ph.desc["page_ids"][pb + lp])] = (r, lp)
    count = np.zeros((plan.n_new, wl.Hkv, n_slots), dtype=np.int32)
    slots_seen = {}
    ps = wl.page_size
    for it in plan.items():
        assert it["n_q_tok"] * wl.G <= (256 if dealt else 64) and it["n_pages"] >= 1 and it["key0"] % ps == 0
        if chunk:
            assert it["n_pages"] * ps <= chunk
        for i in range(int(it["n_q_tok"])):
            tok = int(it["q_tok0"]) + i
            assert treq[tok] == it["request"]
            for pg in range(int(it["n_pages"])):
                e = int(it["page0"]) + pg
                r, lp = where[int(page_ids[e])]
                assert r == it["request"]
                for row in range(int(n_valid[e])):
                    kg = int(it["key0"]) + pg * ps + row
                    other = shared and page_in_branch[e] * ps + row < below[tok]     # shared mask: smaller offset, any branch
                    if kg < pe[tok] or lo[tok] <= kg < hi[tok] or other:
                        count[tok, int(it["kv_head"]), lp * ps + row] += 1
            slots_seen.setdefault((tok, int(it["kv_head"])), []).append(int(it["part_slot"]))
    for h in range(wl.Hkv):
        np.testing.assert_array_equal(count[:, h, :], vis.astype(np.int32))
    # partial slots of a (token, head) are 0 .. n-1, each used once
    for key, sl in slots_seen.items():
        assert sorted(sl) == list(range(len(sl)))
    assert plan.info.n_partials == sum(len(v) for v in slots_seen.values())
    # every listed page has 1..page_size valid rows
    assert ((n_valid >= 1) & (n_valid <= ps)).all()
    if not dealt:       # pages read = pages of the streams
        assert plan.info.kv_tokens_read == int(n_valid.sum())
    return slots_seen


@pytest.mark.parametrize("chunk,n_ctas", [(0, 0), (16, 0), (48, 5), (4096, 1), (0, 1000)])
def test_work_list_covers_every_visible_key_exactly_once(chunk, n_ctas):
    """Integers only, each visible key once, for every phase of the small workloads."""
    for wl in small_workloads():
        for ph in wl.phases:
            plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, chunk_tokens=chunk, n_ctas=n_ctas, host_only=True)
            _check_cover(wl, ph, plan, chunk=chunk)
            plan.destroy()


def test_shared_mask_plans_cover_the_oracles_visible_sets():
    """The visible mask of the ablation: the library's visible sets and the plans' work lists equal
    the oracle's, bit for bit; such plans neither fuse the append nor deal whole streams."""
    for wl in small_workloads():
        for ph in wl.phases:
            n_slots = int(ph.desc["n_pages"].max()) * wl.page_size
            np.testing.assert_array_equal(B.visible_slots(ph.desc, ph.mode, n_slots, mask=B.MASK_SHARED),
                                          oracle.visible_slots(ph.desc, ph.mode, n_slots, mask=oracle.MASK_SHARED))
            for chunk, n_ctas in ((0, 0), (32, 3), (0, 2)):
                plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, chunk_tokens=chunk, n_ctas=n_ctas, host_only=True,
                              mask=B.MASK_SHARED)
                if ph.mode == B.MODE_BRANCH:
                    assert not plan.info.fused_append and not plan.info.direct_output
                _check_cover(wl, ph, plan, chunk=chunk, mask=oracle.MASK_SHARED)
                plan.destroy()
    # pages of 32 rows that are new in full (the page entry's bit fields must not run into each other)
    wl = W.build_segment_workload("p32", 8, 4, 2, 64, "f32", 1e4, [33], [[0, 31, 2]], [[70, 40, 1]], page_size=32)
    ph = wl.phases[-1]
    for mask in (B.MASK_BRANCH_INVISIBLE, B.MASK_SHARED):
        plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, host_only=True, mask=mask)
        _check_cover(wl, ph, plan, mask=mask, dealt=bool(plan.info.direct_output) or plan.info.n_partials == plan.n_new * wl.Hkv)
        plan.destroy()
    assert _plan_rc(W.config_tiny(), W.config_tiny().phases[-1].desc, W.config_tiny().phases[-1].mode, mask=7) == -1     # ASPD_ERR_INVALID_ARG


@pytest.mark.parametrize("kernel,wide_rows", [(B.KERNEL_MMA, 0), (B.KERNEL_MMA, 128), (B.KERNEL_GENERIC, 0)])
def test_dealt_plan_of_a_step_with_many_query_tokens(kernel, wide_rows):
    """Many more streams than CTAs: whole streams are dealt out, one record per (token, head);
    each row block lists the prefix and only the branch pages its tokens see (up to 256 rows, two
    query tiles, for the tensor-core kernel, or 128 when asked), and the visible sets are still
    exactly the oracle's."""
    wl = W.build_segment_workload("deal", 31, 28, 4, 128, "bf16", 1e6, [70, 9, 33], [[0, 17, 5, 2], [3], [0, 0]],
                                  [[40, 25, 31, 1], [21], [2, 50]], serial_steps=0)
    ph = wl.phases[-1]
    plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, kernel=kernel, n_ctas=6, host_only=True, wide_rows=wide_rows)
    items = plan.items()
    assert int(items["n_q_tok"].max()) == ((18 if wide_rows == 128 else 36) if kernel == B.KERNEL_MMA else 9)
    assert plan.info.max_rows_per_item == ((128 if wide_rows == 128 else 256) if kernel == B.KERNEL_MMA else 64)
    assert (items["part_slot"] == 0).all() and (items["key0"] == 0).all()
    seen = _check_cover(wl, ph, plan, dealt=True)
    assert all(len(v) == 1 for v in seen.values())
    first = plan.cta_ranges()
    per_cta = np.diff(first)
    assert per_cta.max() - per_cta.min() <= 1 and per_cta.sum() == len(items)
    # no row block lists a page of a branch that none of its tokens belongs to
    page_ids, n_valid = plan.stream_pages()
    pe, _, _ = plan.token_ranges()
    _, slot, treq = oracle.new_tokens(ph.desc, ph.mode)
    d = ph.desc
    def branch_of(r, s_):
        for b in range(int(d["branch_begin"][r]), int(d["branch_begin"][r]) + int(d["n_branches"][r])):
            if int(d["br_kv_off"][b]) <= s_ < int(d["br_kv_off"][b]) + int(d["br_kv_len"][b]):
                return b
        return -1
    logical = {}
    for r in range(len(d["prefix_len"])):
        for lp in range(int(d["n_pages"][r])):
            logical[int(d["page_ids"][int(d["page_begin"][r]) + lp])] = lp
    for it in items:
        toks = range(int(it["q_tok0"]), int(it["q_tok0"]) + int(it["n_q_tok"]))
        own = {branch_of(int(it["request"]), int(slot[t])) for t in toks}
        for pg in range(int(it["n_pages"])):
            if pg * wl.page_size >= pe[toks[0]]:
                e = int(it["page0"]) + pg
                assert branch_of(int(it["request"]), logical[int(page_ids[e])] * wl.page_size) in own
    plan.destroy()


def test_streams_are_cut_into_equal_shares():
    wl = W.build_segment_workload("cut", 12, 28, 4, 128, "bf16", 1e6, [1000, 300, 2000], [[100, 30], [10], [5, 5, 5]],
                                  [[1, 1], [1], [1, 1, 1]])
    ph = wl.phases[-1]
    for n_ctas in (1, 7, 32):
        plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, n_ctas=n_ctas, host_only=True)
        items = plan.items()
        total = int(items["n_pages"].sum())
        assert total == plan.info.n_stream_pages * wl.Hkv
        assert plan.info.n_ctas == n_ctas
        first = plan.cta_ranges()
        assert first[0] == 0 and first[-1] == len(items) and (np.diff(first) >= 0).all()
        pages = np.array([int(items['n_pages'][first[c]:first[c + 1]].sum()) for c in range(n_ctas)])
        if n_ctas > 1:
            assert pages.max() - pages.min() <= 0.35 * pages.mean() + 16     # cost-balanced, not page-balanced
        # the items, in order, tile the concatenated streams; cutting it into n_ctas contiguous
        # shares of (almost) equal size never needs more than one extra item per share
        assert len(items) <= 3 * wl.Hkv + n_ctas
        plan.destroy()


def test_algorithmic_bytes_formula():
    wl = W.config_qwen7b_layer()
    ph = wl.phases[-1]
    plan = B.Plan(_shape(wl), ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    # each cached token once (prefix 2048 + 4 x 129), K and V, 4 KV heads x 128 x 2 bytes;
    # plus q in / out (28 heads) and the 4 appended tokens
    assert plan.info.kv_tokens_read == 2048 + 4 * 129
    assert plan.info.algorithmic_bytes == 2 * 4 * 128 * 2 * 2564 + 2 * 2 * 28 * 128 * 4 + 2 * 4 * 128 * 2 * 4


def _plan_rc(wl, desc, mode=B.MODE_BRANCH, **kw):
    try:
        B.Plan(_shape(wl), desc, kw.pop("n_pool_pages", wl.n_pool_pages), mode, host_only=True, **kw).destroy()
        return 0
    except B.AspdError as e:
        return e.status


def test_malformed_descriptors_are_rejected_without_launching():
    wl = W.build_segment_workload("v", 6, 4, 2, 64, "f32", 1e4, [20], [[5, 9]], [[1, 1]], serial_steps=1)
    par = [p for p in wl.phases if p.label == "parallel-step"][0]
    good = par.desc
    assert _plan_rc(wl, good) == 0

    def mutated(**kw):
        d = {k: v.copy() for k, v in good.items()}
        for k, (i, val) in kw.items():
            d[k][i] = val
        return d

    BAD = -2
    assert _plan_rc(wl, mutated(br_q_len=(0, 99))) == BAD                 # q_len > kv_len
    assert _plan_rc(wl, mutated(br_kv_off=(1, 33))) == BAD                # not page-aligned
    assert _plan_rc(wl, mutated(br_kv_off=(1, 32))) == BAD                # overlaps branch 0
    assert _plan_rc(wl, mutated(br_kv_len=(1, 4000))) == BAD              # beyond the page table
    assert _plan_rc(wl, mutated(prefix_len=(0, 40))) == BAD               # prefix runs into branch 0
    assert _plan_rc(wl, mutated(prefix_len=(0, -1))) == BAD
    assert _plan_rc(wl, mutated(page_ids=(0, int(good["page_ids"][1])))) == BAD   # duplicate page
    assert _plan_rc(wl, mutated(page_ids=(0, wl.n_pool_pages))) == BAD            # page outside the pool
    assert _plan_rc(wl, good, mode=B.MODE_SERIAL) == BAD                  # serial step without a tail token
    assert _plan_rc(wl, good, mode=7) == -1
    assert _plan_rc(wl, good, chunk_tokens=24) == -1                      # not a multiple of the page size
    bad_shape = B.make_shape(4, 2, 96, 16, "f32", 1e4, 0.1)
    with pytest.raises(B.AspdError) as e:
        B.Plan(bad_shape, good, wl.n_pool_pages, 0, host_only=True)
    assert e.value.status == -3
    assert B.pool_bytes(bad_shape, 4) == 0
    with pytest.raises(B.AspdError) as e:
        B.Plan(B.make_shape(4, 3, 64, 16, "f32", 1e4, 0.1), good, wl.n_pool_pages, 0, host_only=True)
    assert e.value.status == -1
    # the tensor-core kernel is built for bf16 / d 128 / page 16 only
    assert _plan_rc(wl, good, kernel=B.KERNEL_MMA) == -3


def test_rerotation_by_ranges_checks_its_arguments_before_any_launch():
    """aspd_k_rerotate_ranges / _layers validate on the host (nothing here reaches the device): a
    negative count, base or slot, missing or misaligned pools, a negative layer count; no layer and
    no range are valid and do nothing."""
    import ctypes
    L = B.lib()
    sh = B.make_shape(28, 4, 128, 16, "bf16", 1e6, 0.088)
    shp = ctypes.addressof(sh)
    ranges = np.array([[0, 16, 5, 3]], dtype=np.int32)
    table = np.zeros(4, dtype=np.int32)
    fake = ctypes.c_void_p(4096)                     # non-null, 16-byte aligned; never dereferenced on these paths
    pools = (ctypes.c_void_p * 2)(4096, 8192)
    rp, tp = ranges.ctypes.data, table.ctypes.data
    assert L.aspd_k_rerotate_ranges_layers(shp, pools, 0, tp, rp, 1, None) == 0          # no layer
    assert L.aspd_k_rerotate_ranges_layers(shp, pools, 2, tp, rp, 0, None) == 0          # no range
    assert L.aspd_k_rerotate_ranges_layers(shp, pools, -1, tp, rp, 1, None) == -1
    assert L.aspd_k_rerotate_ranges_layers(shp, pools, 2, tp, rp, -1, None) == -1
    assert L.aspd_k_rerotate_ranges_layers(shp, None, 2, tp, rp, 1, None) == -1
    assert L.aspd_k_rerotate_ranges_layers(shp, pools, 2, None, rp, 1, None) == -1
    assert L.aspd_k_rerotate_ranges_layers(shp, (ctypes.c_void_p * 2)(4096, 0), 2, tp, rp, 1, None) == -1     # a missing pool
    assert L.aspd_k_rerotate_ranges_layers(shp, (ctypes.c_void_p * 2)(4096, 8200), 2, tp, rp, 1, None) == -1  # misaligned
    assert L.aspd_k_rerotate_ranges(shp, None, tp, rp, 1, None) == -1
    for bad in ([-1, 16, 5, 3], [0, -16, 5, 3], [0, 16, -5, 3], [0, 2**31 - 4, 8, 3]):
        r = np.array([[0, 0, 0, 9], bad], dtype=np.int32)
        assert L.aspd_k_rerotate_ranges_layers(shp, pools, 2, tp, r.ctypes.data, 2, None) == -2
        assert L.aspd_k_rerotate_ranges(shp, fake, tp, r.ctypes.data, 2, None) == -2
    bad_shape = B.make_shape(4, 2, 96, 16, "f32", 1e4, 0.1)
    assert L.aspd_k_rerotate_ranges_layers(ctypes.addressof(bad_shape), pools, 2, tp, rp, 1, None) == -3


def test_empty_inputs():
    wl = W.build_segment_workload("e", 8, 4, 2, 64, "f32", 1e4, [20], [[5, 9]], [[1, 1]])
    desc = {k: v.copy() for k, v in wl.phases[-1].desc.items()}
    desc["br_q_len"][:] = 0                                  # every branch already finished
    assert B.count_new_tokens(desc, 0) == 0
    plan = B.Plan(_shape(wl), desc, wl.n_pool_pages, 0, host_only=True)
    assert plan.n_new == 0 and plan.info.n_items == 0
    empty = {k: np.zeros(0, np.int32) for k in W.DESC_REQ_KEYS + W.DESC_BR_KEYS + ("page_ids",)}
    assert B.count_new_tokens(empty, 0) == 0
    plan = B.Plan(_shape(wl), empty, 0, 0, host_only=True)
    assert plan.n_new == 0


def test_pool_bytes():
    sh = B.make_shape(28, 4, 128, 16, "bf16", 1e6, 0.088)
    assert B.pool_bytes(sh, 10) == 10 * 4 * 16 * 128 * 2
    sh = B.make_shape(4, 1, 64, 16, "f32", 1e4, 0.125)
    assert B.pool_bytes(sh, 3) == 3 * 1 * 16 * 64 * 4
