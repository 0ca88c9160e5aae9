"""The allocation-free entry point, loki_alloc_solve_static.

Some users of this library may not allocate GPU memory once their process is up:
the serving stack around them has handed the whole device to its own memory pool,
or they sit on a latency-critical path where cudaMalloc's device-wide stall is not
acceptable.  They create the handle at start-up and afterwards call the static
entry point, whose working memory is a fixed array inside the library.

The test calls it through the C-ABI twice in a row with different demand sweeps
(the second call finds the first call's leftovers in the shared array) and wants
byte-identical plans to loki_alloc_solve -- the same bar as the other parity
tests: integers and accuracy bits equal.  It lives in a file pytest collects last
so that a run stopping at the first failure has already run everything else.
"""
import pytest

from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _plans(alloc, n):
    return alloc.torch.clone(alloc.d_out[: n * B.CONFIG_SIZE]).cpu().numpy().tobytes()


def test_static_entry_matches_the_allocating_one_twice_in_a_row():
    import torch
    w = W.make_workload("C2", v=4, n_levels=64)
    sweep_a = list(w.demand_mqps)
    sweep_b = [d // 3 + 7 for d in reversed(w.demand_mqps)][:37]      # shorter, different
    a = B.Allocator(w)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        # the fixed array was bound to the device when the handle was created: the first static
        # call must not make the driver load or allocate anything (a caller whose pool owns the
        # whole GPU could not afford it), so the device's free memory stays what it was
        torch.cuda.synchronize()
        n0 = a.upload(sweep_a)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), n0, stream, a.d_out.data_ptr()) == B.LOKI_OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        for sweep in (sweep_a, sweep_b):
            n = a.upload(sweep)
            a.solve_device(n)                       # existing entry point (direct kernel)
            torch.cuda.synchronize()
            want = _plans(a, n)
            a.d_out.zero_()
            rc = B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), n, stream, a.d_out.data_ptr())
            assert rc == B.LOKI_OK
            torch.cuda.synchronize()
            got = _plans(a, n)
            assert got == want
            plans = B._parse(got, n)
            assert any(p.status == B.LOKI_LEVEL_FEASIBLE for p in plans)
    finally:
        a.close()


def test_static_entry_rejects_what_does_not_fit_its_fixed_array():
    import torch
    w = W.make_workload("C2", v=3, n_levels=80)
    a = B.Allocator(w)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        a.upload(w.demand_mqps)
        torch.cuda.synchronize()
        rc = B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), 65, stream, a.d_out.data_ptr())
        assert rc == B.LOKI_ERR_RANGE and "range" in B.loki_alloc_strerror(rc)
        assert B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), 0, stream,
                                         a.d_out.data_ptr()) == B.LOKI_ERR_INVALID_ARG
        assert B.loki_alloc_solve_static(None, a.d_demand.data_ptr(), 1, stream,
                                         a.d_out.data_ptr()) == B.LOKI_ERR_INVALID_ARG
        # 64 levels is the largest accepted size
        assert B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), 64, stream,
                                         a.d_out.data_ptr()) == B.LOKI_OK
        torch.cuda.synchronize()
    finally:
        a.close()
