"""Shared test plumbing: move seeded workloads to the GPU, run them through the
C-ABI binding, run the oracle, compare with the stated tolerance."""
import numpy as np


def to_device(wl, data, device="cuda:0", fp32=False):
    import torch
    ins = [torch.from_numpy(a).to(device=device, dtype=torch.float32 if fp32 else torch.bfloat16) for a in data["inputs"]]
    ws = []
    for a, kind in zip(data["weights"], wl.weight_kinds):
        dt = torch.float32 if (kind == "bias" or fp32) else torch.bfloat16
        ws.append(torch.from_numpy(a).to(device=device, dtype=dt))
    return ins, ws


def run_gpu(binding, wl, data, mode, device="cuda:0", fp32=False):
    import torch
    sg = binding.Subgraph(wl.ops, wl.input_shapes, mode=mode, dtype=binding.AGO_FP32 if fp32 else binding.AGO_BF16)
    ins, ws = to_device(wl, data, device, fp32)
    out = sg.run(ins, ws)
    torch.cuda.synchronize()
    st = sg.status()
    assert st == binding.AGO_OK, binding.ago_last_error()
    assert tuple(out.shape) == tuple(wl.output_shape)
    res = out.float().cpu().numpy().astype(np.float64)
    sg.close()
    return res


def assert_close(gpu, ref, rel=1e-2, abs_=1e-3, what=""):
    """max |gpu - ref| <= rel * max |ref| + abs_, both maxima over the whole tensor."""
    err = float(np.max(np.abs(gpu - ref)))
    bound = rel * float(np.max(np.abs(ref))) + abs_
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    assert err <= bound, f"{what}: max abs err {err:.4g} > bound {bound:.4g} (max|ref| {np.max(np.abs(ref)):.4g})"
    return err, bound
