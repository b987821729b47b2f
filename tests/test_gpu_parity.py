"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs.  Integer work is compared bit for bit; floating point within the stated bounds:

  bf16 in / fp32 accumulate : max-abs <= 2e-2, mean-abs <= 2e-3  (the acceptance bound), and a
                              tighter relative L2 <= 1e-2 because the absolute bound is of the
                              size of the signal at long contexts
  fp32                      : max-abs <= 1e-4, mean-abs <= 1e-5, relative L2 <= 1e-5
"""
import numpy as np
import pytest

import oracle
from oracle.run import OracleRun, run_workload as oracle_run
from paper_2508_08895_b200 import binding as B, workloads as W

from parity_check import TOL, check, errors

pytestmark = pytest.mark.gpu


def engine():
    from paper_2508_08895_b200 import engine as E
    return E


def compare_workload(wl, **kw):
    ref = oracle_run(wl, kw.get("mask", 0))            # ASPD_MASK_* and the oracle's MASK_* are the same numbers
    run = engine().run_workload(wl, **kw)
    assert len(run.outputs) == len(ref.outputs) and len(ref.outputs) > 0
    for n, (g, r) in enumerate(zip(run.outputs, ref.outputs)):
        check(g, r, wl.dtype, f"{wl.name} output {n}")
    for (p, s, q), (op, os_, oq) in zip(run.positions, ref.positions):
        np.testing.assert_array_equal(p, op)
        np.testing.assert_array_equal(s, os_)
    assert run.cache.canaries_intact(), "a kernel wrote outside the pools"
    return run, ref


KERNELS = [B.KERNEL_GENERIC, B.KERNEL_AUTO]


@pytest.mark.parametrize("kernel", KERNELS)
def test_config1_tiny_fp32(kernel):
    compare_workload(W.config_tiny(), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("theta", [1.0e4, 1.0e6])
def test_config2_qwen7b_layer(kernel, theta):
    compare_workload(W.config_qwen7b_layer(theta=theta), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_config3_branch_open_merge_serial(kernel):
    wl = W.config_branch_open()
    E = engine()
    ref = oracle_run(wl)
    run = E.WorkloadRun(wl, kernel=kernel)
    snap = None
    for ph in wl.phases:
        if ph.label == "serial-0":
            # the merge moved nothing: the pools hold the same bytes as right after the open step
            assert snap is not None
        run.step(ph)
        if ph.label == "parallel-step":
            snap = (run.cache.k.clone(), run.cache.v.clone())
    assert len(run.outputs) == 65
    check(run.outputs[0], ref.outputs[0], wl.dtype, "open step (72 queries)")
    check(np.concatenate(run.outputs[1:]), np.concatenate(ref.outputs[1:]), wl.dtype, "64 serial steps")
    # The merge moved nothing and the serial steps wrote only tail rows: every page outside the tail
    # region holds the bytes it held right after the open step, K and V alike.
    import torch
    d = wl.phases[-1].desc
    first, last = int(d["tail_off"][0]) // wl.page_size, (int(d["tail_off"][0]) + int(d["tail_len"][0]) - 1) // wl.page_size
    tail_pages = set(int(x) for x in d["page_ids"][int(d["page_begin"][0]) + first: int(d["page_begin"][0]) + last + 1])
    assert len(tail_pages) == 4 and int(d["tail_len"][0]) == 64
    keep = torch.tensor([pg not in tail_pages for pg in range(wl.n_pool_pages)], device=run.cache.k.device)
    for now, then in ((run.cache.k, snap[0]), (run.cache.v, snap[1])):
        now, then = now.view(wl.n_pool_pages, -1), then.view(wl.n_pool_pages, -1)
        assert torch.equal(now[keep], then[keep])
        assert (now[~keep] != then[~keep]).any()          # the tail pages are the ones that changed
    for (p, s, q), (op, os_, oq) in zip(run.positions, ref.positions):
        np.testing.assert_array_equal(p, op)
    assert run.positions[-1][0].tolist() == [1024 + 72 + 63]


@pytest.mark.parametrize("kernel", KERNELS)
def test_config4_long_rag(kernel):
    compare_workload(W.config_long_rag(), kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_config5_serving_mix_full_size(kernel):
    """Full size, in the launch configuration the benchmark times (automatic plan)."""
    wl = W.config_serving_mix()
    run, ref = compare_workload(wl, kernel=kernel)
    # Requests with a single branch are plain serial decoding (N = 1): the same tokens through
    # aspd_serial_attn over the same cache -- the branch described as the main branch's tail, so the
    # new token keeps its slot and gets position P + len - 1 either way -- give the same output.
    import torch
    E = engine()
    ph = wl.phases[-1]
    d = ph.desc
    singles = [r for r in range(len(d["prefix_len"])) if d["n_branches"][r] == 1 and d["br_q_len"][d["branch_begin"][r]] == 1]
    assert len(singles) >= 2
    b_of = [int(d["branch_begin"][r]) for r in singles]
    sd = {"prefix_len": d["prefix_len"][singles], "n_branches": np.zeros(len(singles), np.int32),
          "branch_begin": np.zeros(len(singles), np.int32), "page_begin": d["page_begin"][singles], "n_pages": d["n_pages"][singles],
          "tail_off": d["br_kv_off"][b_of], "tail_len": d["br_kv_len"][b_of],
          "br_kv_off": np.zeros(0, np.int32), "br_kv_len": np.zeros(0, np.int32), "br_q_len": np.zeros(0, np.int32),
          "page_ids": d["page_ids"]}
    sd = {k: np.ascontiguousarray(v, dtype=np.int32) for k, v in sd.items()}
    pos_b, _, req_b = B.positions(d, W.MODE_BRANCH)
    rows = [int(np.flatnonzero(req_b == r)[0]) for r in singles]
    pos_s, slot_s, _ = B.positions(sd, W.MODE_SERIAL)
    np.testing.assert_array_equal(pos_s, pos_b[rows])
    plan = B.Plan(run.shape, sd, wl.n_pool_pages, W.MODE_SERIAL, kernel=kernel)
    q = E.to_device(np.ascontiguousarray(ph.q[rows]), wl.dtype)
    out = torch.empty_like(q)
    B.serial_attn(plan, q, run.cache.k, run.cache.v, out)
    torch.cuda.synchronize()
    assert plan.status() == 0
    serial = out.float().cpu().numpy()
    check(serial, ref.outputs[-1][rows], wl.dtype, "single-branch requests through the serial call")
    assert np.abs(serial - run.outputs[-1][rows]).max() <= 1e-2
    plan.destroy()


def test_masked_prefill_full_size():
    """The masked-prefill workload of the benchmark (the serving mix in teacher-forcing layout,
    17 069 query tokens) at full size, in the launch configuration the benchmark times: dealt
    streams, wide row blocks, output written by the attention kernel (fused step call)."""
    wl = W.config_masked_prefill()
    ph = wl.phases[-1]
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    assert plan.info.direct_output and plan.info.max_rows_per_item == 256 and plan.info.n_ctas == 148
    plan.destroy()
    run, ref = compare_workload(wl, fused=True, stable_cache=True)
    assert run.outputs[0].shape[0] == 17069


# Peaked variant: bounds per kernel, about 1.5 x the errors measured on a B200 (recorded with the
# derivation in the design notes): the tensor-core path feeds bf16 K', bf16 rotated Q and bf16
# softmax weights to the MMAs, the generic kernel keeps Q and the weights in fp32.
# Measured: tensor-core kernel max-abs 3.5e-2, mean-abs 2.0e-3, rel-L2 6.0e-3; generic kernel 1.9e-2,
# 1.5e-3, 4.5e-3.
PEAKED_TOL = {B.KERNEL_AUTO: dict(max_abs=5.5e-2, mean_abs=3e-3, rel_l2=9e-3),
              B.KERNEL_GENERIC: dict(max_abs=3e-2, mean_abs=2.4e-3, rel_l2=7e-3)}


@pytest.mark.parametrize("kernel", KERNELS)
def test_peaked_softmax_variant(kernel, record_property):
    """sm_scale x 4: logits ~ N(0, 16), outputs are O(1), so the bounds bite.  The cached keys are
    bf16 on both kernels and, on the tensor-core path, so are the rotated query and the softmax
    weights (relative rounding 2^-9 each) while the oracle keeps everything exact; that perturbs a
    logit of standard deviation 4 by several 1e-3 and an O(1) output by a few 1e-3 on average, a few
    1e-2 at the maximum."""
    wl = W.config_qwen7b_layer()
    wl.sm_scale *= 4.0
    ref = oracle_run(wl)
    run = engine().run_workload(wl, kernel=kernel)
    g, r = run.outputs[0].astype(np.float64), ref.outputs[0]
    assert np.abs(r).max() > 0.5
    mx, mean, rel = errors(g, r)
    print("peaked variant, kernel %d: max-abs %.3e mean-abs %.3e rel-l2 %.3e" % (kernel, mx, mean, rel))
    for k, v in (("max_abs", mx), ("mean_abs", mean), ("rel_l2", rel)):
        record_property(k, v)
    check(g, r, wl.dtype, "peaked", tol=PEAKED_TOL[kernel])


@pytest.mark.parametrize("chunk,n_ctas", [(16, 0), (64, 0), (448, 0), (32768, 0), (16, 3), (0, 1), (48, 37)])
@pytest.mark.parametrize("kernel,combine", [(B.KERNEL_GENERIC, B.COMBINE_AUTO), (B.KERNEL_AUTO, B.COMBINE_KERNEL),
                                            (B.KERNEL_AUTO, B.COMBINE_FUSED)])
def test_split_k_counts_agree(chunk, n_ctas, kernel, combine):
    """Forced cuts of the key streams (every `chunk` keys) and forced grid sizes: one item per page,
    hundreds of items per CTA (beyond what a CTA keeps in shared memory, and more last records per
    CTA than its merge queue holds), a single CTA; records merged by the combine kernel or inside the
    attention kernel."""
    wl = W.config_long_rag(prefix=1024 + 7)
    compare_workload(wl, kernel=kernel, chunk_tokens=chunk, n_ctas=n_ctas, combine=combine)


@pytest.mark.parametrize("fused", [False, True])
def test_merge_inside_the_attention_kernel_gives_the_combine_kernels_bits(fused):
    """a7 by a combine launch and a7 by the last-arriving CTAs of the attention kernel are the same
    arithmetic in the same record order: identical outputs, on the serving mix (stream-K cuts), with
    forced cuts, and on a request whose streams all lie inside one CTA (written without records)."""
    E = engine()
    cases = [(W.config_serving_mix(n_req=8), {}), (W.config_serving_mix(n_req=8), dict(chunk_tokens=160, n_ctas=5)),
             (W.build_segment_workload("one", 31, 28, 4, 128, "bf16", 1e6, [90], [[40, 17]], [[1, 1]], serial_steps=1), {})]
    for wl, kw in cases:
        a = E.run_workload(wl, combine=B.COMBINE_KERNEL, fused=fused, **kw)
        b = E.run_workload(wl, combine=B.COMBINE_FUSED, fused=fused, **kw)
        assert len(a.outputs) == len(b.outputs) > 0
        for x, y in zip(a.outputs, b.outputs):
            np.testing.assert_array_equal(x, y)
        ref = oracle_run(wl)
        for x, r in zip(b.outputs, ref.outputs):
            check(x, r, wl.dtype, wl.name)


@pytest.mark.parametrize("kernel", KERNELS)
def test_ragged_edges(kernel):
    """Lengths that straddle page boundaries, one-token branches, an empty prefix, finished
    branches, several requests."""
    wl = W.build_segment_workload("ragged", 77, 28, 4, 128, "bf16", 1e6, [15, 16, 17, 0, 1, 300],
                                  [[14, 15, 16], [0], [31, 0, 47, 1], [5, 0], [16], [255, 256, 1, 0, 99, 17, 33, 64]],
                                  [[1, 1, 1], [1], [1, 1, 0, 1], [1, 1], [0], [1] * 8], serial_steps=2)
    compare_workload(wl, kernel=kernel)
    wl = W.build_segment_workload("ragged-f32", 78, 4, 2, 64, "f32", 1e4, [15, 33], [[14, 15, 16], [0, 40]],
                                  [[1, 1, 1], [3, 2]], serial_steps=2)
    compare_workload(wl, kernel=kernel)


def test_single_branch_equals_serial_path():
    """N = 1 through aspd_branch_attn equals the same tokens decoded through aspd_serial_attn."""
    E = engine()
    wl = W.build_segment_workload("n1", 9, 28, 4, 128, "bf16", 1e6, [333], [[40]], [[1]])
    a = E.run_workload(wl).outputs[0]
    ph = {p.label: p for p in wl.phases}
    ws = W.build_segment_workload("n1s", 9, 28, 4, 128, "bf16", 1e6, [373], [[]], [[]], serial_steps=1)
    ws.phases[0].k_new[:] = np.concatenate([ph["fill-prefix"].k_new, ph["fill-branches"].k_new])
    ws.phases[0].v_new[:] = np.concatenate([ph["fill-prefix"].v_new, ph["fill-branches"].v_new])
    ws.phases[1].k_new[:] = ph["parallel-step"].k_new
    ws.phases[1].v_new[:] = ph["parallel-step"].v_new
    ws.phases[1].q[:] = ph["parallel-step"].q
    b = E.run_workload(ws).outputs[0]
    ref = oracle_run(wl).outputs[0]
    check(a, ref, "bf16"); check(b, ref, "bf16")
    assert np.abs(a - b).max() <= 1e-2


def test_append_writes_rotated_keys_at_the_mapped_slots():
    E = engine()
    for wl in (W.config_tiny(), W.build_segment_workload("ap", 5, 28, 4, 128, "bf16", 1e6, [17], [[15, 16]], [[1, 1]],
                                                           serial_steps=1)):
        ref = oracle_run(wl)
        run = E.run_workload(wl)
        rel = 2.0 ** -8 if wl.dtype == "bf16" else 1e-6
        n = 0
        for ph, (pos, slot, req) in zip(wl.phases, ref.positions):
            for t in range(0, len(pos), max(1, len(pos) // 40)):
                r = int(req[t]); s = int(slot[t])
                page = int(ph.desc["page_ids"][int(ph.desc["page_begin"][r]) + s // wl.page_size]); row = s % wl.page_size
                for h in range(wl.Hkv):
                    k = run.read_token("k", page, row, h); v = run.read_token("v", page, row, h)
                    np.testing.assert_array_equal(v, ph.v_new[t, h])                 # V is copied bit for bit
                    want = ref.k_pool[page, h, row]
                    assert np.all(np.abs(k - want) <= rel * np.abs(want) + 1e-6), (wl.name, t, h)
                    n += 1
        assert n > 20
        # rows nobody wrote stay zero
        spare = sorted(set(range(wl.n_pool_pages)) - set(wl.phases[-1].desc["page_ids"].tolist()))
        assert spare
        assert not run.read_token("k", spare[0], 3, 0).any()


def _probe(wl, r_digit, n_digits):
    """K = 0 and V = one-hot(digit of the logical slot) in every phase."""
    for ph in wl.phases:
        ph.k_new[:] = 0.0
        ph.v_new[:] = 0.0
    ref = OracleRun(wl)
    for ph in wl.phases:
        pos, slot, req = oracle.new_tokens(ph.desc, ph.mode)
        digit = (slot >> (r_digit * int(np.log2(n_digits)))) & (n_digits - 1)
        ph.v_new[np.arange(len(slot)), :, digit] = 1.0
    return wl


@pytest.mark.parametrize("mask", [B.MASK_BRANCH_INVISIBLE, B.MASK_SHARED])
@pytest.mark.parametrize("kernel", KERNELS)
def test_mask_membership_through_the_kernels_is_exact(kernel, mask):
    """With all keys zero every visible key weighs exactly 1/n; with one-hot V rows the output
    column c is (number of visible keys whose slot digit is c) / n.  The counts recovered from
    the kernels' output equal the oracle's visible sets as integers (fp32), and the zero
    pattern is exact (bf16)."""
    E = engine()
    for dtype, Hq, Hkv, d in (("f32", 4, 2, 64), ("bf16", 28, 4, 128)):
        for r_digit in (0, 1):
            wl = W.build_segment_workload("probe", 55, Hq, Hkv, d, dtype, 1e4, [70, 9], [[14, 15, 16], [200]],
                                          [[2, 1, 3], [1]], serial_steps=1)
            wl = _probe(wl, r_digit, d)
            run = E.run_workload(wl, kernel=kernel, mask=mask)
            outs = iter(run.outputs)
            for ph in wl.phases:
                if not ph.compare:
                    continue
                out = next(outs)
                n_slots = int(ph.desc["n_pages"].max()) * wl.page_size
                vis = oracle.visible_slots(ph.desc, ph.mode, n_slots, mask=mask)
                for t in range(vis.shape[0]):
                    slots = np.flatnonzero(vis[t])
                    digit = (slots >> (r_digit * int(np.log2(d)))) & (d - 1)
                    want = np.bincount(digit, minlength=d)
                    n = len(slots)
                    for h in range(Hq):
                        got = out[t, h].astype(np.float64) * n
                        np.testing.assert_array_equal(got == 0, want == 0)
                        if dtype == "f32":
                            np.testing.assert_array_equal(np.rint(got).astype(np.int64), want)
                            assert np.abs(got - want).max() < 1e-3
                        else:
                            assert np.abs(got - want).max() <= 0.01 * max(want.max(), 1)


def test_branch_permutation_permutes_outputs_on_gpu():
    E = engine()
    prior, newq = [70, 33, 129], [1, 1, 1]
    wl = W.build_segment_workload("p", 4, 28, 4, 128, "bf16", 1e6, [500], [prior], [newq])
    base = E.run_workload(wl).outputs[0]
    ph = {p.label: p for p in wl.phases}
    perm = [2, 0, 1]
    cuts = np.concatenate([[0], np.cumsum(prior)])
    wp = W.build_segment_workload("p2", 4, 28, 4, 128, "bf16", 1e6, [500], [[prior[i] for i in perm]], [newq])
    pp = {p.label: p for p in wp.phases}
    pp["fill-prefix"].k_new[:] = ph["fill-prefix"].k_new; pp["fill-prefix"].v_new[:] = ph["fill-prefix"].v_new
    pp["fill-branches"].k_new[:] = np.concatenate([ph["fill-branches"].k_new[cuts[i]:cuts[i + 1]] for i in perm])
    pp["fill-branches"].v_new[:] = np.concatenate([ph["fill-branches"].v_new[cuts[i]:cuts[i + 1]] for i in perm])
    for name in ("k_new", "v_new", "q"):
        getattr(pp["parallel-step"], name)[:] = getattr(ph["parallel-step"], name)[perm]
    outp = E.run_workload(wp).outputs[0]
    assert np.abs(outp - base[perm]).max() <= 2e-3


def test_step_host_matches_device_path():
    import torch
    E = engine()
    wl = W.config_qwen7b_layer()
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode)
    pos, _, _ = B.positions(ph.desc, ph.mode)
    q = E.to_device(ph.q, wl.dtype).cpu().pin_memory()
    k = E.to_device(ph.k_new, wl.dtype).cpu().pin_memory()
    v = E.to_device(ph.v_new, wl.dtype).cpu().pin_memory()
    out = torch.empty_like(q).pin_memory()
    B.step_host(plan, q, k, v, np.ascontiguousarray(pos), run.cache.k, run.cache.v, out)
    host = out.float().numpy()
    dev = run.step(ph)
    np.testing.assert_array_equal(host, dev)
    check(host, oracle_run(wl).outputs[0], wl.dtype)
    # the asynchronous form: two plans on two streams (as two layers of a model would), one wait at the end
    plan_b = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode)
    outs = [torch.zeros_like(q).pin_memory() for _ in range(4)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    pos_h = torch.from_numpy(np.ascontiguousarray(pos)).pin_memory()
    torch.cuda.synchronize()
    for i, o in enumerate(outs):
        B.step_host_async((plan, plan_b)[i & 1], q, k, v, pos_h, run.cache.k, run.cache.v, o, stream=streams[i & 1])
    for st in streams:
        st.synchronize()
    for o in outs:
        np.testing.assert_array_equal(o.float().numpy(), dev)
    assert plan.status() == 0 and plan_b.status() == 0
    # q, k_new, v_new packed into one host buffer: a single copy carries them
    packed = torch.cat([q.reshape(-1), k.reshape(-1), v.reshape(-1)]).pin_memory()
    nq, nk = q.numel(), k.numel()
    out_p = torch.zeros_like(q).pin_memory()
    B.step_host(plan, packed[:nq], packed[nq:nq + nk], packed[nq + nk:], pos_h, run.cache.k, run.cache.v, out_p)
    np.testing.assert_array_equal(out_p.float().numpy(), dev)
    # position IDs that are not the plan's (a position-ID variant for the keys): they are copied and
    # the append kernel uses them -- same result as aspd_kv_append + aspd_branch_attn on the device
    pos5 = np.ascontiguousarray(pos + 5)
    out_v = torch.zeros_like(q).pin_memory()
    B.step_host(plan, q, k, v, pos5, run.cache.k, run.cache.v, out_v)
    out_d = torch.empty_like(q, device="cuda")
    B.kv_append(plan, k.cuda(), v.cuda(), torch.from_numpy(pos5).cuda(), run.cache.k, run.cache.v)
    B.branch_attn(plan, q.cuda(), run.cache.k, run.cache.v, out_d)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out_v.float().numpy(), out_d.float().cpu().numpy())
    assert np.abs(out_v.float().numpy() - dev).max() > 1e-3
    plan.destroy(); plan_b.destroy()


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    """A wait nothing satisfies runs into its limit (about a millisecond here), reports
    ASPD_ERR_TIMEOUT, and the device keeps working afterwards."""
    import time
    import torch
    t0 = time.perf_counter()
    assert B.debug_bounded_wait(2_000_000) == -5
    assert time.perf_counter() - t0 < 5.0
    x = torch.arange(8, device="cuda")
    assert int(x.sum().item()) == 28
    compare_workload(W.config_tiny())


@pytest.mark.parametrize("kernel", KERNELS)
def test_fused_step_appends_and_attends_like_the_two_calls(kernel):
    """aspd_branch_step / aspd_serial_step: same outputs within tolerance, and the rows they write
    into the cache are the rotated keys and raw values the oracle's append produces."""
    E = engine()
    for wl in (W.build_segment_workload("fs", 41, 28, 4, 128, "bf16", 1e6, [15, 300, 0], [[14, 15, 16], [255, 1, 99], [3]],
                                        [[1, 1, 1], [1, 0, 1], [1]], serial_steps=2),
               W.config_branch_open(serial_steps=2), W.config_tiny()):
        ref = oracle_run(wl)
        run = E.run_workload(wl, kernel=kernel, fused=True)
        assert len(run.outputs) == len(ref.outputs)
        for g, r in zip(run.outputs, ref.outputs):
            check(g, r, wl.dtype, wl.name)
        rel = 2.0 ** -8 if wl.dtype == "bf16" else 1e-6
        for ph, (pos, slot, req) in zip(wl.phases, ref.positions):
            if ph.q is None:
                continue
            for t in range(0, len(pos), max(1, len(pos) // 12)):
                r = int(req[t]); s_ = int(slot[t])
                page = int(ph.desc["page_ids"][int(ph.desc["page_begin"][r]) + s_ // wl.page_size]); row = s_ % wl.page_size
                for h in range(wl.Hkv):
                    np.testing.assert_array_equal(run.read_token("v", page, row, h), ph.v_new[t, h])
                    want = ref.k_pool[page, h, row]
                    got = run.read_token("k", page, row, h)
                    assert np.all(np.abs(got - want) <= rel * np.abs(want) + 1e-6)


@pytest.mark.parametrize("fused", [False, True])
def test_stable_cache_promise_changes_nothing_but_timing(fused):
    """With aspd_tuning_t.stable_cache the producers fetch pages that hold no new rows before the
    previous kernel on the stream has finished; results are the same."""
    for wl in (W.config_serving_mix(n_req=6), W.config_branch_open(serial_steps=3)):
        run, ref = compare_workload(wl, fused=fused, stable_cache=True)
        base = engine().run_workload(wl, fused=fused)
        for a, b in zip(run.outputs, base.outputs):
            np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("fused", [False, True])
def test_second_parallel_stage(kernel, fused):
    """Iterative serial/parallel switching: branches of a second stage see the prefix, the merged
    branches of the first stage and the serial tokens between the stages (regions with
    q_len = ASPD_Q_SHARED), plus their own branch; positions continue from the complete sequence."""
    for wl in (W.build_two_stage_workload("ts", 5, 28, 4, 128, "bf16", 1e6, 700, [130, 1, 47], 5, [33, 0, 140, 16],
                                          [1, 1, 1, 1], serial_steps=2),
               W.build_two_stage_workload("ts-open", 6, 28, 4, 128, "bf16", 1e6, 90, [20, 31], 0, [0, 0, 0], [12, 12, 12],
                                          serial_steps=1),
               W.build_two_stage_workload("ts-f32", 7, 4, 1, 64, "f32", 1e4, 33, [9, 16], 2, [3, 7], [1, 1], serial_steps=1)):
        run, ref = compare_workload(wl, kernel=kernel, fused=fused)
        assert len(run.outputs) == 1 + sum(p.label.startswith("serial") for p in wl.phases)


@pytest.mark.parametrize("rule", ["fix-k", "same-max"])
@pytest.mark.parametrize("fused", [False, True])
def test_position_id_variants(rule, fused):
    """The ablation's position-ID variants (pre-allocated fixed-length intervals per branch;
    Same-Max) are plain caller-given positions for the library: aspd_kv_append's `pos` and the
    plan's `q_pos`."""
    from test_oracle_pins import _variant_positions
    E = engine()
    wl = W.build_segment_workload("var", 17, 28, 4, 128, "bf16", 1e6, [700], [[130, 2, 47, 64]], [[1, 1, 1, 1]], serial_steps=2)
    variant = _variant_positions(wl, rule)
    ref = OracleRun(wl)
    run = E.WorkloadRun(wl, fused=fused)
    for ph, pos in zip(wl.phases, variant):
        ref.step(ph, pos_override=pos)
        run.step(ph, pos_override=pos)
    assert len(run.outputs) == 3
    for g, r in zip(run.outputs, ref.outputs):
        check(g, r, "bf16", rule)
    plain = oracle_run(wl)
    assert np.abs(plain.outputs[-1] - ref.outputs[-1]).max() > 1e-3     # the variant really differs from Eq. 4


@pytest.mark.parametrize("mma_m", [64, 96, 128])
def test_mma_m_variants_on_the_decode_shapes(mma_m):
    """The tensor-core kernel's stream-K path with M = 128 MMAs (rows replicated to fill the
    accumulator) and with M = 64 (half the tensor work, accumulators in 16 lanes of each quadrant,
    two rows per softmax thread): the serving mix (row blocks of 7 to 56 rows: both padded sizes,
    one and two replicas), ragged edges, forced cuts with many items per CTA, a single CTA, the
    visible mask, the fused step, a second stage and serial steps, at the default scale and with
    logits x 4 (references raised along the stream: the long way of a tile, with O rescaled)."""
    E = engine()
    wl = W.config_serving_mix(n_req=12)
    run, ref = compare_workload(wl, mma_m=mma_m)
    compare_workload(wl, mma_m=mma_m, fused=True, stable_cache=True)
    ph = wl.phases[-1]
    plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, mma_m=mma_m, host_only=True)
    assert plan.info.mma_m == mma_m and not plan.info.dealt
    rows = plan.items()["n_q_tok"] * 7
    assert (rows <= 32).any() and (rows > 32).any()
    plan.destroy()
    rag = W.build_segment_workload("ragged", 77, 28, 4, 128, "bf16", 1e6, [15, 16, 17, 0, 1, 300],
                                   [[14, 15, 16], [0], [31, 0, 47, 1], [5, 0], [16], [255, 256, 1, 0, 99, 17, 33, 64]],
                                   [[1, 1, 1], [1], [1, 1, 0, 1], [1, 1], [0], [1] * 8], serial_steps=2)
    compare_workload(rag, mma_m=mma_m)
    compare_workload(rag, mma_m=mma_m, mask=B.MASK_SHARED)
    lr = W.config_long_rag(prefix=1024 + 7)
    for chunk, n_ctas in ((16, 0), (448, 0), (0, 1), (48, 37)):
        compare_workload(lr, mma_m=mma_m, chunk_tokens=chunk, n_ctas=n_ctas)
    two = W.build_two_stage_workload("ts", 61, 28, 4, 128, "bf16", 1e6, 200, [30, 5, 41], 3, [17, 0, 6], [1, 1, 1], serial_steps=2)
    compare_workload(two, mma_m=mma_m, fused=True)
    peaked = W.config_qwen7b_layer()
    peaked.sm_scale *= 4.0
    ref = oracle_run(peaked)
    run = E.run_workload(peaked, mma_m=mma_m)
    check(run.outputs[0], ref.outputs[0], "bf16", "peaked", tol=PEAKED_TOL[B.KERNEL_AUTO])
    # logits x 16: along a key stream exponents pass 2^40 against the reference of the item's first
    # tile, so tiles are redone the long way and O is rescaled in tensor memory (in the layout of this
    # variant's P.V).  The softmax is close to an argmax and bf16 keys decide between near-equal
    # candidates differently from the oracle's exact ones for some rows: only gross errors are excluded.
    peaked.sm_scale *= 4.0
    for wl16 in (peaked, W.config_long_rag(prefix=4096 + 5)):
        if wl16 is not peaked:
            wl16.sm_scale *= 16.0
        ref = oracle_run(wl16)
        run = E.run_workload(wl16, mma_m=mma_m)
        g_, r_ = run.outputs[0].astype(np.float64), ref.outputs[0]
        err = np.abs(g_ - r_)
        assert np.isfinite(g_).all() and err.mean() <= 3e-2, (wl16.name, err.mean())
        assert (err.reshape(err.shape[0], -1).max(axis=1) <= 0.1).mean() >= 0.7, wl16.name
    # A jump built into the keys: from slot 1000 on every key has 96 in the slowest rotary pair's first
    # element and every query 4 (both exact in bf16, hardly rotated), i.e. logits 49 powers of two
    # above the earlier ones.  With two CTAs an item has many tiles, the jump falls into a later tile of
    # one: its sum passes 2^40, the tile is redone the long way, the reference raised and O rescaled.
    jump = W.config_long_rag(prefix=2048 + 5)
    for ph in jump.phases:
        if ph.label == "fill-prefix":
            ph.k_new[1000:, :, 63] = 96.0
        if ph.q is not None:
            ph.q[:, :, 63] = 4.0
    compare_workload(jump, mma_m=mma_m, n_ctas=2)
    compare_workload(jump, mma_m=mma_m, n_ctas=2, fused=True)
    # open step of config 3: 72 query tokens in row blocks of 9 (63 rows), several blocks per request
    compare_workload(W.config_branch_open(serial_steps=2), mma_m=mma_m)


@pytest.mark.parametrize("combine", [B.COMBINE_KERNEL, B.COMBINE_FUSED])
def test_deterministic_across_repeated_launches(combine):
    """Repeated launches of the same step give bit-identical outputs (no data race in the
    warp-specialised pipeline shows up as run-to-run noise), whether a combine launch merges the
    records or the attention kernel's last-arriving CTAs do (whichever CTA that is, the records are
    merged in record order)."""
    import torch
    E = engine()
    wl = W.config_serving_mix(n_req=8)
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, stable_cache=True, combine=combine)
    assert plan.info.single_launch == (1 if combine == B.COMBINE_FUSED else 0)
    q, k, v = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    outs = [torch.empty_like(q) for _ in range(6)]
    first = None
    for _ in range(10):
        for o in outs:
            B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, o)
        torch.cuda.synchronize()
        for o in outs:
            first = o.clone() if first is None else first
            assert torch.equal(o, first)
    assert plan.status() == 0


@pytest.mark.parametrize("kernel", KERNELS)
def test_masked_prefill_of_a_parallel_segment(kernel):
    """Many query tokens per branch in one step (block-diagonal across branches, causal inside a
    branch, over a shared prefix): 240 query tokens = 27 row blocks that each stream the keys."""
    wl = W.build_segment_workload("prefill", 29, 28, 4, 128, "bf16", 1e6, [300, 40], [[0, 17, 5], [0]],
                                  [[100, 60, 31], [49]], serial_steps=1)
    run, ref = compare_workload(wl, kernel=kernel)
    assert run.outputs[0].shape[0] == 240
    # with few CTAs the plan has many more streams than CTAs and deals whole streams instead of
    # cutting; the tensor-core kernel then runs its variants for such plans: row blocks of two
    # query tiles (up to 36 tokens), or of one tile (18 tokens) when asked
    compare_workload(wl, kernel=kernel, n_ctas=8)
    compare_workload(wl, kernel=kernel, n_ctas=8, wide_rows=128)


@pytest.mark.parametrize("wide_rows", [128, 256])
def test_wide_row_blocks_mixed_sizes_and_raised_maxima(wide_rows):
    """The variants of the tensor-core kernel for dealt plans, on row blocks of 1 to 18 tokens (one
    query tile: 7 to 126 rows, all three softmax layouts in one launch) or 1 to 36 tokens (two query
    tiles, the second absent, partly or completely filled), tiles with padding rows, requests
    whose only visible keys are their own, at the default scale and with logits x 4 (the reference
    maximum of a row is raised many times along its key stream; bounds derived as for the peaked
    decode variant)."""
    E = engine()
    wl = W.build_segment_workload("wide", 37, 28, 4, 128, "bf16", 1e6, [700, 33, 0, 129], [[0, 40, 3], [5], [0, 0], [200]],
                                  [[130, 9, 4], [1], [20, 3], [57]], serial_steps=1)
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    ph = [x for x in wl.phases if x.mode == W.MODE_BRANCH and x.q is not None][-1]
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, n_ctas=5, host_only=True, wide_rows=wide_rows)
    ntok = plan.items()["n_q_tok"]
    if wide_rows == 128:
        assert ntok.max() == 18 and ntok.min() <= 4 and ((ntok > 4) & (ntok <= 9)).any()
    else:
        assert plan.info.max_rows_per_item == 256 and ntok.max() == 36 and ntok.min() == 1 and ((ntok > 18) & (ntok < 36)).any()
    plan.destroy()
    compare_workload(wl, n_ctas=5, wide_rows=wide_rows)
    compare_workload(wl, n_ctas=5, fused=True, wide_rows=wide_rows)
    wl.sm_scale *= 4.0
    ref = oracle_run(wl)
    run = E.run_workload(wl, n_ctas=5, wide_rows=wide_rows)
    g, r = run.outputs[0].astype(np.float64), ref.outputs[0]
    err = np.abs(g - r)
    assert err.max() <= 6e-2 and err.mean() <= 4e-3
    # logits x 16: exponents pass 2^40 along a row's key stream, where the two-tile variant raises its
    # reference (the one-tile variants raise theirs at 2^8 and did so above already).  The softmax is
    # close to an argmax here and the bf16 keys decide between near-equal candidates differently from
    # the oracle's exact ones for some rows, so only gross errors are excluded: finite, a loose mean
    # bound, and most rows agree closely.
    wl.sm_scale *= 4.0
    ref = oracle_run(wl)
    run = E.run_workload(wl, n_ctas=5, wide_rows=wide_rows)
    g, r = run.outputs[0].astype(np.float64), ref.outputs[0]
    err = np.abs(g - r)
    assert np.isfinite(g).all() and err.mean() <= 3e-2
    assert (err.reshape(err.shape[0], -1).max(axis=1) <= 0.1).mean() >= 0.8
    assert np.linalg.norm(g - r) / np.linalg.norm(r) <= 1e-2


@pytest.mark.parametrize("n_ctas", [1, 2, 7])
def test_two_tile_row_blocks_at_their_edges(n_ctas):
    """The two-tile variant where its bookkeeping changes: requests with exactly 18, 19, 35, 36, 37 and
    73 query tokens (a second tile that is absent, holds one token, is one short of full, full; a
    block boundary crossed by one token; three blocks), an empty prefix, key streams of 1 to 9+
    pages (tiles whose second half has no keys), and a single CTA that walks more items than it
    caches in shared memory, so that the second group sits out whole runs of items."""
    wl = W.build_segment_workload("w2edge", 59, 28, 4, 128, "bf16", 1e6, [0, 3, 70, 129, 16, 250, 40],
                                  [[0], [1], [0, 0], [5], [0, 2], [0, 9, 0], [0, 0, 0, 0]],
                                  [[18], [19], [35, 1], [36], [37, 3], [73, 2, 20], [1, 2, 18, 19]], serial_steps=1)
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    ph = [x for x in wl.phases if x.mode == W.MODE_BRANCH and x.q is not None][-1]
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, n_ctas=n_ctas, host_only=True)
    items = plan.items()
    assert plan.info.dealt and plan.info.max_rows_per_item == 256 and plan.info.n_ctas == n_ctas
    assert {4, 18, 19, 23, 36}.issubset(set(int(x) for x in items["n_q_tok"]))
    assert int(np.diff(plan.cta_ranges()).max()) > 8 or n_ctas > 2
    plan.destroy()
    compare_workload(wl, n_ctas=n_ctas)
    compare_workload(wl, n_ctas=n_ctas, fused=True, stable_cache=True)


def test_two_tile_plain_pass_with_huge_and_tiny_exponents():
    """The two-tile variant's common pass takes a quarter of its exponentials as a cubic with the
    exponent bits patched in (keys 6, 7, 14, 15 of every page) and judges an overflow from the sum.
    Prefix keys scaled by 400 at such places, deep inside the prefix (full, unmasked halves): for some
    rows their logits are far above 2^127 relative to the reference (the clamp keeps the patched
    exponent in range, the sum shows the overflow, the reference is raised), for others far below
    2^-126 (weights that must vanish, not wrap around).  A row whose jump is positive puts nearly
    all its weight on that key, so the output is close to that key's V row."""
    E = engine()
    wl = W.build_segment_workload("w2jump", 67, 28, 4, 128, "bf16", 1e6, [600, 300, 400], [[0, 5], [3], [0]], [[30, 25], [36], [20]])
    fill = [p for p in wl.phases if p.label == "fill-prefix"][0]
    # one scaled key per request (two would tie for some rows, and a tie between logits of several
    # hundred is decided by the bf16 rounding of the cached keys): slots 310 and 150 take the cubic,
    # slot 305 the special-function unit
    for slot in (310, 600 + 150, 900 + 305):
        fill.k_new[slot] *= 400.0
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    ph = [x for x in wl.phases if x.label == "parallel-step"][0]
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, n_ctas=3, host_only=True)
    assert plan.info.dealt and plan.info.max_rows_per_item == 256
    plan.destroy()
    ref = oracle_run(wl)
    for n_ctas in (3, 1):
        run = E.run_workload(wl, n_ctas=n_ctas)
        g, r = run.outputs[0].astype(np.float64), ref.outputs[0]
        err = np.abs(g - r)
        assert np.isfinite(g).all()
        # A cached key 400 times the usual size carries 400 times the usual rounding error (several
        # units of its logit), so a row for which the scaled key's logit falls within ten units of its
        # other keys' largest puts a different weight on it than the oracle does (up to all or none:
        # errors of the size of a V row).  Those rows are about 1 %.  A wrapped exponent or a missed
        # overflow spoils the many rows whose scaled key is hundreds of units above or below everything
        # else (measured with the upper clamp taken out: mean error 1.2e-2 instead of 8e-4, 97.6 %
        # of the rows within 3e-2 instead of 99.0 %; without the lower clamp: not finite).
        row_err = err.reshape(-1, err.shape[-1]).max(axis=1)
        assert (row_err <= 3e-2).mean() >= 0.985 and err.mean() <= 2e-3, ((row_err <= 3e-2).mean(), err.max(), err.mean())


def test_large_decode_batch_takes_the_dealt_plan():
    """A decode step with many more (request, KV head) streams than CTAs: whole streams are dealt
    out, the append is still fused into the attention launch (few new rows per CTA), the kernel
    writes the output itself, and every item has at most 3 x 7 rows (the narrow softmax layouts
    inside the wide kernel)."""
    rng = np.random.default_rng(3)
    prefix = [int(x) for x in rng.integers(20, 400, size=10)]
    prior = [[int(x) for x in rng.integers(1, 60, size=int(rng.integers(1, 4)))] for _ in prefix]
    wl = W.build_segment_workload("big", 53, 28, 4, 128, "bf16", 1e6, prefix, prior, [[1] * len(p) for p in prior], serial_steps=1)
    ph = [x for x in wl.phases if x.mode == W.MODE_BRANCH and x.q is not None][-1]
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, n_ctas=8, host_only=True)
    assert plan.info.direct_output and plan.info.fused_append and plan.info.n_items == 40
    plan.destroy()
    for fused in (True, False):
        compare_workload(wl, n_ctas=8, fused=fused, stable_cache=fused)


def test_wide_row_blocks_with_very_negative_logits():
    """All logits near -130 in log2 units (keys and queries opposite along the slowest rotary pair,
    so the rotation hardly changes them): against the wide variant's initial reference of 0 every
    weight would underflow to 0; the reference has to come down to the row's first keys.  The
    softmax is then close to uniform and the output the mean of the visible V rows."""
    wl = W.build_segment_workload("neg", 41, 28, 4, 128, "bf16", 1e6, [130, 20], [[0, 7], [0]], [[40, 22], [30]])
    for ph in wl.phases:
        ph.k_new[:] = 0.0
        ph.k_new[:, :, 63] = 32.0
        if ph.q is not None:
            ph.q[:] = 0.0
            ph.q[:, :, 63] = -32.0
    run, ref = compare_workload(wl, n_ctas=3)
    assert np.abs(ref.outputs[0]).max() < 1.0 and run.outputs[0].shape[0] == 92


def test_rerotation_moves_cached_keys_to_new_positions():
    """Same-Re without a re-prefill: after a segment, the branch tokens are renumbered
    sequentially by rotating their cached keys by (new - old) positions in place."""
    import torch
    E = engine()
    for wl in (W.build_segment_workload("re", 19, 28, 4, 128, "bf16", 1e6, [40], [[17, 3, 30]], [[1, 1, 1]]), W.config_tiny()):
        run = E.run_workload(wl)
        ref = oracle_run(wl)
        d = wl.phases[-1].desc
        P = int(d["prefix_len"][0])
        pages, rows, delta, want = [], [], [], []
        at = P                                         # sequential renumbering: branch after branch
        for b in range(int(d["n_branches"][0])):
            for k in range(int(d["br_kv_len"][b])):
                s_ = int(d["br_kv_off"][b]) + k
                pages.append(int(d["page_ids"][s_ // wl.page_size])); rows.append(s_ % wl.page_size)
                delta.append(at - (P + k)); at += 1
        t = lambda x: torch.tensor(x, dtype=torch.int32, device="cuda")
        before = [run.read_token("k", pg, r, 0) for pg, r in zip(pages, rows)]
        vbefore, kbefore = run.cache.v.clone(), run.cache.k.clone()
        B.k_rerotate(run.shape, run.cache.k, t(pages), t(rows), t(delta))
        torch.cuda.synchronize()
        assert torch.equal(run.cache.v, vbefore)
        # the same renumbering given as one range per branch (table base, first slot, count, delta): same bytes
        ranges, before_b = [], 0
        for b in range(int(d["n_branches"][0])):
            ranges.append((0, int(d["br_kv_off"][b]), int(d["br_kv_len"][b]), before_b))
            before_b += int(d["br_kv_len"][b])
        k2 = kbefore.clone()
        B.k_rerotate_ranges(run.shape, k2, t(d["page_ids"].tolist()), np.array(ranges + [(0, 5, 0, 99)], dtype=np.int32))
        torch.cuda.synchronize()
        assert torch.equal(k2, run.cache.k) and not torch.equal(k2, kbefore)
        assert run.cache.canaries_intact()
        # Two roundings to the storage dtype: the stored key is off by half an ulp of each element,
        # the rotation mixes the pair (i, i + d/2), and the result is rounded again.
        ulp_half = 2.0 ** -8 if wl.dtype == "bf16" else 4e-6    # bf16: 8 significand bits
        moved = 0
        for (pg, r, dl, old) in zip(pages, rows, delta, before):
            for h in range(wl.Hkv):
                got = run.read_token("k", pg, r, h)
                want = oracle.rope(ref.k_pool[pg, h, r], float(dl), wl.theta)     # = RoPE(k, new position)
                pair = np.hypot(want[:wl.d // 2], want[wl.d // 2:])
                bound = 1.05 * ulp_half * (np.sqrt(2.0) * np.tile(pair, 2) + np.abs(want)) + 1e-7
                assert np.all(np.abs(got - want) <= bound), (pg, r, h, float(np.max(np.abs(got - want) / bound)))
            moved += int(dl != 0 and not np.array_equal(run.read_token("k", pg, r, 0), old))
        assert moved > 0


def test_same_re_serial_decoding_after_rerotation():
    """The paper's Same-Re variant end to end: after the segment the branch tokens get sequential
    position IDs (keys re-rotated in place), then serial decoding continues over the merged cache.
    The oracle rotates its own fp64 keys by the same offsets (RoPE composition, pinned on the CPU)."""
    import torch
    E = engine()
    wl = W.build_segment_workload("same-re", 23, 28, 4, 128, "bf16", 1e6, [70, 33], [[20, 9, 31], [5, 40]],
                                  [[1, 1, 1], [1, 1]], serial_steps=2)
    run, ref = E.WorkloadRun(wl), OracleRun(wl)
    serial = [i for i, ph in enumerate(wl.phases) if ph.mode == W.MODE_SERIAL]
    for ph in wl.phases[:serial[0]]:
        run.step(ph); ref.step(ph)
    d = wl.phases[serial[0] - 1].desc
    pages, rows, delta = [], [], []
    for r in range(len(d["prefix_len"])):
        P, at = int(d["prefix_len"][r]), int(d["prefix_len"][r])
        pg0 = int(d["page_begin"][r])
        for b in range(int(d["branch_begin"][r]), int(d["branch_begin"][r]) + int(d["n_branches"][r])):
            for k in range(int(d["br_kv_len"][b])):
                s_ = int(d["br_kv_off"][b]) + k
                pages.append(int(d["page_ids"][pg0 + s_ // wl.page_size])); rows.append(s_ % wl.page_size)
                delta.append(at - (P + k)); at += 1
    t = lambda x: torch.tensor(x, dtype=torch.int32, device="cuda")
    # one range per branch; every request has its own page table inside the concatenated one
    ranges = []
    for r in range(len(d["prefix_len"])):
        moved = 0
        for b in range(int(d["branch_begin"][r]), int(d["branch_begin"][r]) + int(d["n_branches"][r])):
            ranges.append((int(d["page_begin"][r]), int(d["br_kv_off"][b]), int(d["br_kv_len"][b]), moved))
            moved += int(d["br_kv_len"][b])
    check_k = run.cache.k.clone()
    # three layers' pools (different contents, the same page tables) in one launch against one call each
    layers = [run.cache.k.clone(), (run.cache.k.float() * 0.5).to(run.cache.k.dtype), run.cache.k.flip(0).contiguous()]
    singles = [x.clone() for x in layers]
    B.k_rerotate(run.shape, check_k, t(pages), t(rows), t(delta))
    B.k_rerotate_ranges(run.shape, run.cache.k, t(d["page_ids"].tolist()), np.array(ranges, dtype=np.int32))
    B.k_rerotate_ranges_layers(run.shape, layers, t(d["page_ids"].tolist()), np.array(ranges, dtype=np.int32))
    for x in singles:
        B.k_rerotate_ranges(run.shape, x, t(d["page_ids"].tolist()), np.array(ranges, dtype=np.int32))
    B.k_rerotate_ranges_layers(run.shape, [], t(d["page_ids"].tolist()), np.array(ranges, dtype=np.int32))    # no layer: nothing
    torch.cuda.synchronize()
    assert torch.equal(check_k, run.cache.k) and torch.equal(layers[0], check_k)
    assert all(torch.equal(a, b) for a, b in zip(layers, singles)) and not torch.equal(layers[1], layers[0])
    for pg, r, dl in zip(pages, rows, delta):
        for h in range(wl.Hkv):
            ref.k_pool[pg, h, r] = oracle.rope(ref.k_pool[pg, h, r], float(dl), wl.theta)
    assert max(delta) > 0
    for i in serial:                        # the serial position P + sum(len) is already sequential
        got, want = run.step(wl.phases[i]), ref.step(wl.phases[i])
        check(got, want, wl.dtype, "same-re serial step")


def test_rerotation_by_ranges_in_several_launches():
    """More ranges than one launch carries (512) and more pools than one launch carries (64): 603
    single-token ranges over 70 pools in one call give the bits of three whole-branch ranges applied
    to a pool by itself.  (The ranges of one call must not overlap: every key is read and written once.)"""
    import torch
    E = engine()
    wl = W.build_segment_workload("re-many", 29, 28, 4, 128, "bf16", 1e6, [16], [[200, 200, 200]], [[1, 1, 1]])
    run = E.run_workload(wl)
    d = wl.phases[-1].desc
    t = lambda x: torch.tensor(x, dtype=torch.int32, device="cuda")
    table = t(d["page_ids"].tolist())
    whole, moved = [], 0
    for b in range(3):
        whole.append((0, int(d["br_kv_off"][b]), int(d["br_kv_len"][b]), moved))
        moved += int(d["br_kv_len"][b])
    single = [(base, s0 + i, 1, dl) for (base, s0, n, dl) in whole for i in range(n)]
    assert len(single) == 603
    want = run.cache.k.clone()
    B.k_rerotate_ranges(run.shape, want, table, np.array(whole, dtype=np.int32))
    pools = [run.cache.k.clone() for _ in range(70)]
    B.k_rerotate_ranges_layers(run.shape, pools, table, np.array(single, dtype=np.int32))
    torch.cuda.synchronize()
    assert not torch.equal(want, run.cache.k)
    assert all(torch.equal(x, want) for x in pools)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("kernel", KERNELS)
def test_shared_mask_variant(kernel, fused):
    """The visible mask of the paper's attention-mask ablation (a token at offset k also sees the
    first k tokens of the other branches of its stage): decode steps over branches of different
    lengths, one of which decodes nothing; a second parallel stage; whole branches in one step;
    split-K cuts inside other branches' regions.  The result differs from the paper's mask."""
    assert oracle.MASK_SHARED == B.MASK_SHARED
    decode = W.build_segment_workload("sh", 43, 28, 4, 128, "bf16", 1e6, [300, 40], [[20, 9, 131, 4], [5, 40]],
                                      [[1, 1, 1, 0], [1, 1]], serial_steps=1)
    two = W.build_two_stage_workload("sh2", 44, 28, 4, 128, "bf16", 1e6, 90, [30, 1, 17], 3, [5, 0, 40], [1, 2, 1], serial_steps=1)
    whole = W.build_segment_workload("sh3", 45, 28, 4, 128, "bf16", 1e6, [100], [[0, 17, 5]], [[40, 25, 31]])
    for wl in (decode, two, whole):
        run, ref = compare_workload(wl, kernel=kernel, fused=fused, mask=B.MASK_SHARED)
        iso = oracle_run(wl)
        assert max(np.abs(a - b).max() for a, b in zip(ref.outputs, iso.outputs)) > 1e-2
    compare_workload(decode, kernel=kernel, fused=fused, mask=B.MASK_SHARED, chunk_tokens=32, n_ctas=5)
    small = W.config_tiny()
    compare_workload(small, kernel=B.KERNEL_GENERIC, fused=fused, mask=B.MASK_SHARED)


def test_misaligned_device_buffers_are_refused_before_any_launch():
    """Buffers are moved in 16-byte pieces; a pointer off that boundary gets ASPD_ERR_INVALID_ARG
    (no kernel runs, the context stays usable and the next call is correct)."""
    import torch
    E = engine()
    wl = W.build_segment_workload("al", 47, 28, 4, 128, "bf16", 1e6, [40], [[17, 3]], [[1, 1]])
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode)
    q, k, v = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    out = torch.empty_like(q)
    def off(t):                                   # same values, storage shifted by one element (2 bytes)
        buf = torch.empty(t.numel() + 8, dtype=t.dtype, device=t.device)
        view = buf[1:1 + t.numel()].view(t.shape)
        view.copy_(t)
        return view
    calls = [lambda: B.branch_step(plan, off(q), k, v, run.cache.k, run.cache.v, out),
             lambda: B.branch_step(plan, q, off(k), v, run.cache.k, run.cache.v, out),
             lambda: B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, off(out)),
             lambda: B.branch_attn(plan, off(q), run.cache.k, run.cache.v, out),
             lambda: B.attn_partials(plan, off(q), run.cache.k, run.cache.v)]
    for call in calls:
        with pytest.raises(B.AspdError) as e:
            call()
        assert e.value.status == -1
    B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, out)
    torch.cuda.synchronize()
    assert plan.status() == 0
    ref = oracle_run(wl)
    check(E.to_host_f32(out), ref.outputs[0], wl.dtype, "after refused calls")
    plan.destroy()


def test_plan_per_step_reuses_device_blocks_without_synchronising():
    """A plan per step, destroyed while its work may still be in flight and on alternating streams:
    the block of a destroyed plan is reused only after the streams it was used on have passed its
    work (events, no host synchronisation), free device memory stays flat, every result is right."""
    import torch
    E = engine()
    wl = W.config_serving_mix(n_req=8)
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    q, k, v = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    ref_plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode)
    ref = torch.empty_like(q)
    B.branch_step(ref_plan, q, k, v, run.cache.k, run.cache.v, ref)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [torch.zeros_like(q) for _ in range(30)]
    B.release_cached_memory()
    free0 = None
    for i, o in enumerate(outs):
        st = streams[i % 3]
        plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, stream=st, n_ctas=[0, 37, 148][i % 3])
        B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, o, stream=st)
        plan.destroy()                             # not waited for
        if i == 8:
            free0 = torch.cuda.mem_get_info()[0]
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free0 - (1 << 20)      # no growth once the first blocks are parked
    want = ref.float().cpu().numpy()
    for i, o in enumerate(outs):
        got = o.float().cpu().numpy()
        if i % 3 == 0:
            np.testing.assert_array_equal(got, want)              # same plan options: same bits
        else:
            assert np.abs(got - want).max() <= 2e-2
    check(outs[-1].float().cpu().numpy(), oracle_run(wl).outputs[0], wl.dtype)
    ref_plan.destroy()
    B.release_cached_memory()


def test_plan_update_in_place_keeps_a_captured_graph_valid():
    """A decode loop over 12 steps: the step (fused append + attention + combine) is captured into a
    CUDA graph once with an updatable plan; every following step calls aspd_plan_update with the
    longer branches and replays the graph.  Each step's output equals that of a fresh plan."""
    import torch
    E = engine()
    n_steps = 12
    prefix, prior = [300, 40, 700], [[20, 9, 131], [5], [64, 3]]
    wl = W.build_segment_workload("upd", 61, 28, 4, 128, "bf16", 1e6, prefix, [[x + n_steps - 1 for x in p] for p in prior],
                                  [[1] * len(p) for p in prior])
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    q, k, v = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    descs = []
    for t in range(n_steps):
        d = {kk: vv.copy() for kk, vv in ph.desc.items()}
        d["br_kv_len"] = (ph.desc["br_kv_len"] - (n_steps - 1 - t)).astype(np.int32)
        descs.append(d)
    k2, v2 = run.cache.k.clone(), run.cache.v.clone()          # a second cache for the fresh plans
    stream = torch.cuda.Stream()
    out_g, out_f = torch.zeros_like(q), torch.zeros_like(q)
    with torch.cuda.stream(stream):
        # a grid size that stays the same while the lengths grow (a full-size step has the whole GPU at every length)
        plan = B.Plan(run.shape, descs[0], wl.n_pool_pages, ph.mode, updatable=True, stable_cache=True, stream=stream, n_ctas=8)
        B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, out_g, stream=stream)     # warm-up outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            B.branch_step(plan, q, k, v, run.cache.k, run.cache.v, out_g, stream=stream)
        for t in range(n_steps):
            if t > 0:
                plan.update(descs[t], stream=stream)
            graph.replay()
            stream.synchronize()
            fresh = B.Plan(run.shape, descs[t], wl.n_pool_pages, ph.mode, stream=stream, n_ctas=8)
            B.branch_step(fresh, q, k, v, k2, v2, out_f, stream=stream)
            stream.synchronize()
            assert plan.status(stream) == 0 and fresh.status(stream) == 0
            np.testing.assert_array_equal(out_g.float().cpu().numpy(), out_f.float().cpu().numpy())
            fresh.destroy()
    assert torch.equal(run.cache.k, k2) and torch.equal(run.cache.v, v2)
    # a step that needs another launch sequence is refused and leaves the plan as it was
    other = {kk: vv.copy() for kk, vv in descs[-1].items()}
    other["br_q_len"] = other["br_q_len"].copy(); other["br_q_len"][0] = 0
    with pytest.raises(B.AspdError) as e:
        plan.update(other, stream=stream)
    assert e.value.status == -3                     # ASPD_ERR_UNSUPPORTED
    with torch.cuda.stream(stream):
        graph.replay()
        stream.synchronize()
    np.testing.assert_array_equal(out_g.float().cpu().numpy(), out_f.float().cpu().numpy())
    plan.destroy()


def test_zero_new_tokens_is_a_no_op():
    E = engine()
    wl = W.build_segment_workload("e", 8, 28, 4, 128, "bf16", 1e6, [20], [[5, 9]], [[1, 1]])
    run = E.run_workload(wl)
    desc = {k: v.copy() for k, v in wl.phases[-1].desc.items()}
    desc["br_q_len"][:] = 0
    plan = B.Plan(run.shape, desc, wl.n_pool_pages, 0)
    assert plan.n_new == 0
    B.kv_append(plan, None, None, None, run.cache.k, run.cache.v)
    B.branch_attn(plan, None, run.cache.k, run.cache.v, None)
    assert plan.status() == 0
