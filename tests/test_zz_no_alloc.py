"""cleave_assemble_static, the assembly entry point for callers that cannot allocate device memory
(processes that have given all of it to their own pool, or loops that cannot afford the stall of a
cudaMalloc): its tables live in a fixed array inside the library instead of buffers allocated on
first use.  It must give exactly what cleave_assemble gives, call after call, although every call
reuses the same array.  Collected last on purpose: a failure here cannot hide the other tests."""
import gc

import numpy as np
import pytest

import cleave_inputs as ci
from helpers import GpuRun, lib_plan_for

pytestmark = pytest.mark.gpu


def _both_ways(w, **opts):
    import torch
    p = lib_plan_for(w, **opts)
    run = GpuRun(w, ci.make_tensors(w), p)
    run.exec()
    run.assemble()                                   # existing entry point (allocates its tables)
    p.check_status()
    ref = run.results()
    out = [torch.full_like(c, float("nan")) for c in run.C]
    p.assemble_static(run.partials, out)             # fixed-array entry point
    torch.cuda.synchronize()
    for g, a, b in zip(w.gemms, ref, out):
        assert np.array_equal(a.view(np.uint32), b.cpu().numpy().view(np.uint32)), g.name
    return p, run


def test_two_calls_in_a_row_match_cleave_assemble():
    # first call: several K-slices and slice-count classes; second call: a different, smaller plan
    # whose tables overwrite only the front of the array the first call filled
    p1, run1 = _both_ways(ci.config(2, 4), kslice_max=512)
    assert max(p1.ksplit(i) for i in range(p1.n_gemms)) >= 2
    _both_ways(ci.config(1))
    # and the first plan again, after its tables were overwritten
    import torch
    out = [torch.full_like(c, float("nan")) for c in run1.C]
    p1.assemble_static(run1.partials, out)
    torch.cuda.synchronize()
    for a, b in zip(run1.results(), out):
        assert np.array_equal(a.view(np.uint32), b.cpu().numpy().view(np.uint32))


def test_no_device_memory_is_taken_by_the_call():
    """The property in the entry point's name: a plan that has never touched the device is assembled
    through the fixed array, and neither the driver's free-memory figure nor torch's allocator moves."""
    import torch
    import paper_2512_22142_b200 as cl
    w = ci.config(2, 4)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w, kslice_max=512)
    run = GpuRun(w, ts, p)
    run.exec(); run.assemble(); p.check_status()
    ref = run.results()
    warm = lib_plan_for(ci.config(1))                       # first use of the array on this device, if it is the first
    x = torch.zeros(warm.arena_elems, dtype=torch.float32, device="cuda:0")
    warm.assemble_static(x, [torch.zeros(256, 768, dtype=torch.float32, device="cuda:0")])
    fresh = lib_plan_for(w, kslice_max=512)                 # same plan, host tables only: no device state yet
    out = [torch.full_like(c, float("nan")) for c in run.C]
    torch.cuda.synchronize()
    # (tensors of earlier tests that only the garbage collector can free are freed now, and the collector rests
    # during the call: the figures below must not move for reasons that are not the call's)
    gc.collect()
    gc.disable()
    try:
        free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        fresh.assemble_static(run.partials, out)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    finally:
        gc.enable()
    for g, a, b in zip(w.gemms, ref, out):
        assert np.array_equal(a.view(np.uint32), b.cpu().numpy().view(np.uint32)), g.name
    # two calls back to back on one stream, nothing in between: the second call's tables wait for the first's kernels
    out2 = [torch.full_like(c, float("nan")) for c in run.C]
    fresh.assemble_static(run.partials, out)
    fresh.assemble_static(run.partials, out2)
    torch.cuda.synchronize()
    for a, b in zip(ref, out2):
        assert np.array_equal(a.view(np.uint32), b.cpu().numpy().view(np.uint32))
    # after a fused execution part of the result sits in the C that execution was given: another C is refused
    run.exec_fused()
    with pytest.raises(cl.CleaveError) as e:
        p.assemble_static(run.partials, out)
    assert e.value.code == -1
    p.assemble_static(run.partials, run.C)
    for a, b in zip(ref, run.results()):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_oversized_plan_is_refused_before_any_launch():
    import paper_2512_22142_b200 as cl
    p = lib_plan_for(ci.config(3))                   # ~3 MiB of tables: beyond the fixed array
    with pytest.raises(cl.CleaveError) as e:
        p.assemble_static(256, [256] * p.n_gemms)    # never dereferenced: refused on size alone
    assert e.value.code == -11
    assert "scratch" in cl.strerror(-11)
