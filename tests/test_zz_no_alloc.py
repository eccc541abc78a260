"""metok_segment_events_static: the entry point for callers that cannot allocate.

Hosts that run inside a fixed memory budget, or that may not trigger the implicit
synchronisation of an allocation where they need the result, cannot hand the library
a workspace.  This entry point uses a 1 MiB array built into the library instead.  It
must give exactly what metok_segment_events gives (same kernels, so bit for bit), on
two calls in a row (the array keeps the previous call's contents), whether this file
runs alone in a fresh process or after every other test (it is collected last)."""

import numpy as np
import pytest
import torch

from paper_2506_02850_b200 import binding as B
from paper_2506_02850_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _same(a, b):
    for key in ("sims", "boundaries", "event_offsets", "frame_event"):
        assert torch.equal(a[key], b[key]), key


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    cfg = W.CONFIGS["frames32"]
    V = torch.from_numpy(W.vision_inputs(cfg)["V"]).to(torch.bfloat16).cuda()
    want = B.metok_segment_events(V, cfg.k)
    first = B.metok_segment_events_static(V, cfg.k)
    torch.cuda.synchronize()
    _same(first, want)
    # second call, other data and shape, on the same array: stale partial sums must not leak in
    rng = np.random.default_rng(5)
    V2 = torch.from_numpy(rng.standard_normal((19, 50, 264)).astype(np.float32)).cuda()
    want2 = B.metok_segment_events(V2, 6)
    second = B.metok_segment_events_static(V2, 6)
    torch.cuda.synchronize()
    _same(second, want2)
    # and the first problem again, plus the token-averaging mode
    _same(B.metok_segment_events_static(V, cfg.k), want)
    _same(B.metok_segment_events_static(V2, 6, B.SIM_MEANPOOL), B.metok_segment_events(V2, 6, B.SIM_MEANPOOL))
    torch.cuda.synchronize()


def test_static_scratch_rejects_problems_beyond_its_capacity():
    cap = B.lib().metok_segment_events_static_capacity()
    assert cap == 1 << 20
    T, N, d = 4096, 1024, 1024                                 # 128 slabs x 4096 frames x 8 bytes = 4 MiB
    need = B.lib().metok_segment_events_workspace_bytes(B.BF16, T, N, d, B.SIM_FLATTEN)
    assert need > cap
    V = torch.zeros((8, 4, 8), dtype=torch.bfloat16, device="cuda")   # pointers are valid, sizes are not read
    sims = torch.empty(T, dtype=torch.float32, device="cuda")
    ints = torch.empty(T + 2, dtype=torch.int32, device="cuda")
    st = B.lib().metok_segment_events_static(V.data_ptr(), B.BF16, T, N, d, 2, B.SIM_FLATTEN, sims.data_ptr(),
                                             ints.data_ptr(), ints.data_ptr(), ints.data_ptr(), None)
    assert st == -6
    assert b"capacity" in B.lib().metok_status_string(st)


def test_static_entry_point_allocates_nothing():
    """The raw C call with outputs allocated beforehand: neither the driver's free-memory figure nor
    torch's allocator moves across it (the device address of the built-in array is already known
    after a first call)."""
    rng = np.random.default_rng(6)
    T, N, d, k = 24, 36, 128, 5
    V = torch.from_numpy(rng.standard_normal((T, N, d)).astype(np.float32)).cuda()
    want = B.metok_segment_events(V, k)
    B.metok_segment_events_static(V, k)                        # first call on this device, if none came before
    sims = torch.empty(T - 1, dtype=torch.float32, device="cuda")
    bnd = torch.empty(k - 1, dtype=torch.int32, device="cuda")
    offs = torch.empty(k + 1, dtype=torch.int32, device="cuda")
    fe = torch.empty(T, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    st = B.lib().metok_segment_events_static(V.data_ptr(), B.F32, T, N, d, k, B.SIM_FLATTEN, sims.data_ptr(),
                                             bnd.data_ptr(), offs.data_ptr(), fe.data_ptr(),
                                             torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert st == 0
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert torch.equal(sims, want["sims"]) and torch.equal(bnd, want["boundaries"])
    assert torch.equal(offs, want["event_offsets"]) and torch.equal(fe, want["frame_event"])
