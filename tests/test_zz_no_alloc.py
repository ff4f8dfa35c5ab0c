"""The entry point that allocates nothing (`tl3_spmm_static_scratch`), collected last.

Some users of the library cannot hand it a workspace because they may not allocate device memory
where they call it (a plug-in's execute hook, a process whose device-memory budget is already
spent).  For them the library keeps 3 MiB of scratch inside its own image.  This test calls that
entry point through the C ABI twice in a row and compares both results with what the regular
`tl3_spmm` (caller-supplied workspace) returns for the same inputs; it also checks that a problem
that needs more scratch than the built-in array is refused instead of launched.
"""
import numpy as np
import pytest

from paper_2607_08786_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_the_regular_one(oracle_mod):
    import torch
    from paper_2607_08786_b200 import build, tl3
    build.build_library()
    L = tl3.lib()
    # 8 row-tiles x 40 k-tiles: every row-tile is shared by many CTAs, so the scratch (partial
    # sums, arrival flags) is really used
    case = wl.Case(0, "static", 1024, 5120, 16, 321, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    m.upload()
    Xd = torch.from_numpy(X).cuda()
    ws = m.new_workspace(case.N)
    Y_ref = m.spmm(Xd, workspace=ws)
    torch.cuda.synchronize()
    assert m.status(ws) == tl3.OK
    assert m.workspace_bytes(case.N) <= tl3.STATIC_SCRATCH_BYTES
    ref = Y_ref.cpu().numpy()
    Yref64, bound = oracle_mod.dense_fp64(W, X)
    tol = oracle_mod.tolerance(bound)
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):                                   # two calls in a row share the array
        Y = torch.full((case.M, case.N), float("nan"), dtype=torch.float16, device="cuda")
        rc = L.tl3_spmm_static_scratch(m._h, Xd.data_ptr(), Xd.stride(0), Y.data_ptr(), Y.stride(0), case.N, stream)
        assert rc == tl3.OK, L.tl3_strerror(rc)
        torch.cuda.synchronize()
        assert L.tl3_static_scratch_status(stream) == tl3.OK
        got = Y.cpu().numpy()
        assert np.all(np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= tol), f"call {call}"
        assert np.all(np.abs(got.astype(np.float64) - Yref64) <= tol), f"call {call}"
        # same kernel, same fixed summation order: the bits agree as well
        assert np.array_equal(got.view(np.uint16), ref.view(np.uint16)), f"call {call}"
    # and it really obtains no device memory: after the warm-up calls above, one more call with Y
    # already allocated leaves the device's free memory and torch's own books where they were
    Y = torch.empty((case.M, case.N), dtype=torch.float16, device="cuda")
    torch.cuda.synchronize()
    free_before, booked_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    rc = L.tl3_spmm_static_scratch(m._h, Xd.data_ptr(), Xd.stride(0), Y.data_ptr(), Y.stride(0), case.N, stream)
    assert rc == tl3.OK
    torch.cuda.synchronize()
    # (>=: memory that an earlier test handed back may still be on its way to the free pool)
    assert torch.cuda.mem_get_info()[0] >= free_before and torch.cuda.memory_allocated() == booked_before


def test_static_scratch_refuses_what_does_not_fit():
    import torch
    from paper_2607_08786_b200 import build, tl3
    build.build_library()
    L = tl3.lib()
    case = wl.Case(0, "big", 256, 256, 64, 5, 0.5, "magnitude")
    m = tl3.encode(case.make_W())
    m.upload()
    X = torch.zeros((256, 64), dtype=torch.float16, device="cuda")
    Y = torch.full((256, 64), 7.0, dtype=torch.float16, device="cuda")
    assert m.workspace_bytes(64) > tl3.STATIC_SCRATCH_BYTES     # 2 slots x SMs x 64 x 128 floats
    rc = L.tl3_spmm_static_scratch(m._h, X.data_ptr(), 64, Y.data_ptr(), 64, 64, torch.cuda.current_stream().cuda_stream)
    assert rc == tl3.ERR_SCRATCH_LIMIT
    assert b"scratch" in L.tl3_strerror(rc)
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())                               # nothing was launched
    with pytest.raises(tl3.Tl3Error):
        m.spmm_static_scratch(X)
