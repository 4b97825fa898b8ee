"""ago_subgraph_run_static: the unfused run for callers that cannot allocate
device memory (a plug-in inside a server with fixed pools, a sandbox without
cudaMalloc after start-up). Its scratch is a 4 MiB array inside the library, so
here it is called through the C-ABI twice in a row and compared with the
ordinary entry point, which takes a caller-allocated workspace. Collected last
on purpose: a failure here cannot hide a failure of any other test."""
import numpy as np
import pytest

from paper_2212_01005_b200 import workloads as WL
from helpers import to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["per_mini_subgraph", "per_op"])
def test_static_scratch_matches_caller_workspace_on_two_calls(ago, mode):
    import torch
    wl = WL.get("mbv2_14")
    data = WL.generate(wl)
    ins, ws = to_device(wl, data)
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode=mode)
    assert 0 < sg.workspace_bytes <= ago.AGO_STATIC_SCRATCH_BYTES
    ref = sg.run(ins, ws)                       # existing entry point, workspace from torch
    torch.cuda.synchronize()
    ref64 = ref.float().cpu().numpy().astype(np.float64)
    bound = 1e-2 * float(np.max(np.abs(ref64))) + 1e-3
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        out = torch.full_like(ref, float("nan"))
        st = ago.ago_subgraph_run_static(sg._h, [t.data_ptr() for t in ins], [t.data_ptr() for t in ws],
                                         [out.data_ptr()], stream)
        assert st == ago.AGO_OK, ago.ago_last_error()
        torch.cuda.synchronize()
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert float(np.max(np.abs(got - ref64))) <= bound, (mode, call)
        assert torch.equal(out, ref), (mode, call)     # same kernels, same order: bit-identical
    sg.close()


def test_static_scratch_rejects_what_does_not_fit(ago):
    import torch
    wl = WL.get("mbv2_56", batch=4)              # intermediates of 3.6 MB each: 2 x 3.6 > 4 MiB
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode="per_mini_subgraph")
    assert sg.workspace_bytes > ago.AGO_STATIC_SCRATCH_BYTES
    dummy = torch.zeros(64, device="cuda:0")
    ptrs = [dummy.data_ptr()] * 8
    assert ago.ago_subgraph_run_static(sg._h, ptrs, ptrs, ptrs, 0) == ago.AGO_ERR_WORKSPACE
    assert "scratch" in ago.ago_last_error()[1]
    sg.close()
    wl = WL.Workload("dw", [5], [(1, 6, 6, 8)], [("conv2d", dict(O=8, R=3, S=3, stride=1, pad=1, groups=8))], samples=1)
    fused = ago.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    assert ago.ago_subgraph_run_static(fused._h, ptrs, ptrs, ptrs, 0) == ago.AGO_ERR_UNSUPPORTED
    fused.close()
