"""aspd_attn_static: the attention of a step with all scratch memory inside an array that is
part of the library, for callers that are not allowed to allocate device memory (a process
whose device memory is owned by a pool, a serving loop that must not re-enter an allocator).

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  The test needs nothing from the other tests and passes alone in a fresh process.
"""
import numpy as np
import pytest

from oracle.run import run_workload as oracle_run
from paper_2508_08895_b200 import binding as B, workloads as W
from parity_check import check

pytestmark = pytest.mark.gpu


def _setup(wl):
    """Fill the cache of one layer through the ordinary path; return what the last phase needs."""
    import torch
    from paper_2508_08895_b200 import engine as E
    run = E.WorkloadRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph)
    ph = wl.phases[-1]
    plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode)
    pos, _, _ = B.positions(ph.desc, ph.mode)
    B.kv_append(plan, E.to_device(ph.k_new, wl.dtype), E.to_device(ph.v_new, wl.dtype),
                torch.from_numpy(pos.copy()).cuda(), run.cache.k, run.cache.v)
    q = E.to_device(ph.q, wl.dtype)
    ref = torch.empty_like(q)
    (B.branch_attn if ph.mode == W.MODE_BRANCH else B.serial_attn)(plan, q, run.cache.k, run.cache.v, ref)
    torch.cuda.synchronize()
    assert plan.status() == 0
    return run, ph, q, ref


@pytest.mark.parametrize("make", [
    lambda: W.config_qwen7b_layer(),
    lambda: W.config_tiny(),
    lambda: W.build_segment_workload("ragged", 77, 28, 4, 128, "bf16", 1e6, [15, 300], [[14, 15, 16], [255, 1, 99]],
                                     [[1, 1, 1], [1, 1, 1]], serial_steps=1),
])
def test_static_scratch_entry_point_matches_the_allocating_one_twice_in_a_row(make):
    """Two calls in a row (the second finds the first one's contents in the array) against the
    allocating entry point and against the oracle, with the bounds of the other parity tests; and
    the calls take no device memory: the driver's count of free bytes does not go down."""
    import torch
    wl = make()
    want_oracle = oracle_run(wl).outputs[-1]
    run, ph, q, ref = _setup(wl)
    host_plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    outs_d = [torch.full_like(q, float("nan")) for _ in range(3)]
    B.attn_static(host_plan, q, run.cache.k, run.cache.v, outs_d[2])      # first call on the device: the array's module is loaded
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for i in range(2):                      # the array keeps the previous call's contents
        B.attn_static(host_plan, q, run.cache.k, run.cache.v, outs_d[i])
        assert B.static_status() == 0
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before          # what cudaMalloc inside the library would take shows here
    outs = [o.float().cpu().numpy() for o in outs_d[:2]]
    want = ref.float().cpu().numpy()
    for got in outs:
        check(got, want.astype(np.float64), wl.dtype, "static against the allocating entry point")
        check(got, want_oracle, wl.dtype, "static against the oracle")
    np.testing.assert_array_equal(outs[0], outs[1])


def test_static_scratch_refuses_a_capturing_stream():
    """The call copies its tables from host memory that lives only as long as the call, so on a
    stream that is being captured it enqueues nothing and says so."""
    import torch
    wl = W.build_segment_workload("cap", 3, 28, 4, 128, "bf16", 1e6, [40], [[5, 9]], [[1, 1]])
    run, ph, q, ref = _setup(wl)
    host_plan = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    out = torch.full_like(q, float("nan"))
    B.attn_static(host_plan, q, run.cache.k, run.cache.v, out)             # set-up call, outside capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            rc = B.lib().aspd_attn_static(host_plan._h, q.data_ptr(), run.cache.k.data_ptr(), run.cache.v.data_ptr(), out.data_ptr(),
                                          torch.cuda.current_stream().cuda_stream)
    assert rc == -3
    torch.cuda.synchronize()
    check(out.float().cpu().numpy(), ref.float().cpu().numpy().astype(np.float64), wl.dtype)


def test_static_scratch_rejects_plans_beyond_its_size_and_device_plans():
    import torch
    wl = W.build_segment_workload("big", 5, 28, 4, 128, "bf16", 1e6, [16384], [[40] * 8], [[1] * 8])
    ph = wl.phases[-1]
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    # 16-key items: thousands of partial records, far more than the 8 MiB array holds
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, chunk_tokens=16, host_only=True)
    dummy = torch.zeros(8 * 28 * 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.AspdError) as e:
        B.attn_static(plan, dummy, dummy, dummy, dummy)
    assert e.value.status == -7
    dev_plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode)
    with pytest.raises(B.AspdError) as e:
        B.attn_static(dev_plan, dummy, dummy, dummy, dummy)
    assert e.value.status == -1


def test_static_scratch_runs_the_plans_other_regimes():
    """Host-only plans made for the wide kernel variant (whole streams dealt, 128-row blocks) and
    for the visible mask of the ablation run through the scratch array like any other."""
    import torch
    wl = W.build_segment_workload("prefill", 29, 28, 4, 128, "bf16", 1e6, [300, 40], [[0, 17, 5], [0]], [[100, 60, 31], [49]])
    run, ph, q, ref = _setup(wl)
    want = ref.float().cpu().numpy()
    wide = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, n_ctas=8, host_only=True)
    assert wide.info.max_rows_per_item == 256
    out = torch.full_like(q, float("nan"))
    B.attn_static(wide, q, run.cache.k, run.cache.v, out)
    torch.cuda.synchronize()
    check(out.float().cpu().numpy(), want.astype(np.float64), "bf16", "wide plan through the scratch array")
    check(out.float().cpu().numpy(), oracle_run(wl).outputs[-1], "bf16", "wide plan against the oracle")
    shared_dev = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, mask=B.MASK_SHARED)
    ref2 = torch.empty_like(q)
    B.branch_attn(shared_dev, q, run.cache.k, run.cache.v, ref2)
    shared_host = B.Plan(run.shape, ph.desc, wl.n_pool_pages, ph.mode, mask=B.MASK_SHARED, host_only=True)
    out2 = torch.full_like(q, float("nan"))
    B.attn_static(shared_host, q, run.cache.k, run.cache.v, out2)
    torch.cuda.synchronize()
    a, b = out2.float().cpu().numpy().astype(np.float64), ref2.float().cpu().numpy().astype(np.float64)
    check(a, b, "bf16", "visible mask through the scratch array")
    check(a, oracle_run(wl, B.MASK_SHARED).outputs[-1], "bf16", "visible mask against the oracle")
    assert np.abs(b - want).max() > 1e-2          # the other mask really is another result
