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


GUARD_BYTES = 8192        # guard band before and after the output and the workspace
GUARD_BYTE = 0xA5


def run_gpu(binding, wl, data, mode, device="cuda:0", fp32=False):
    """One run through the C-ABI. The output and the workspace sit between guard bands filled with a byte pattern
    that is checked after the run: a kernel that stores before the start or past the end of either fails here
    (compute-sanitizer is not available on the test machines, so this is the bounds check)."""
    import torch
    sg = binding.Subgraph(wl.ops, wl.input_shapes, mode=mode, dtype=binding.AGO_FP32 if fp32 else binding.AGO_BF16)
    ins, ws = to_device(wl, data, device, fp32)
    esz = 4 if fp32 else 2
    nbytes = int(np.prod(wl.output_shape)) * esz
    obuf = torch.full((nbytes + 2 * GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device=device)
    out = obuf[GUARD_BYTES:GUARD_BYTES + nbytes].view(torch.float32 if fp32 else torch.bfloat16).view(wl.output_shape)
    need = sg.workspace_bytes
    wbuf = None
    if need:
        wbuf = torch.full((need + 2 * GUARD_BYTES + 256,), GUARD_BYTE, dtype=torch.uint8, device=device)
        base = (wbuf.data_ptr() + GUARD_BYTES + 255) & ~255
        woff = base - wbuf.data_ptr()
        st = binding.ago_subgraph_set_workspace(sg._h, base, need)
        assert st == binding.AGO_OK, binding.ago_last_error()
        sg._ws = wbuf            # keeps the buffer alive and tells the wrapper a workspace is attached
    sg.run(ins, ws, out=out)
    torch.cuda.synchronize()
    st = sg.status()
    assert st == binding.AGO_OK, binding.ago_last_error()
    assert tuple(out.shape) == tuple(wl.output_shape)
    assert bool((obuf[:GUARD_BYTES] == GUARD_BYTE).all()) and bool((obuf[GUARD_BYTES + nbytes:] == GUARD_BYTE).all()), \
        f"{wl.name}/{mode}: a kernel wrote outside the output tensor"
    if wbuf is not None:
        assert bool((wbuf[:woff] == GUARD_BYTE).all()) and bool((wbuf[woff + need:] == GUARD_BYTE).all()), \
            f"{wl.name}/{mode}: a kernel wrote outside the workspace"
    res = out.float().cpu().numpy().astype(np.float64)
    sg.close()
    return res


def rounding_share(oracle, wl, data, ref):
    """Diagnostic only: max |ref - ref_rounded| where ref_rounded rounds the tensors read by the second and later
    complex operators to bf16 (what a bf16 tensor-core pipeline must do). Printed beside a parity error to tell
    rounding noise from a defect; never the pass/fail reference."""
    rr = oracle.run_chain(wl.ops, data["inputs"], data["weights"], round_intermediates_to_bf16=True)
    return float(np.max(np.abs(rr - ref)))


def assert_close(gpu, ref, rel=1e-2, abs_=1e-3, what=""):
    """max |gpu - ref| <= rel * max |ref| + abs_, both maxima over the whole tensor."""
    err = float(np.max(np.abs(gpu - ref)))
    bound = rel * float(np.max(np.abs(ref))) + abs_
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    assert err <= bound, f"{what}: max abs err {err:.4g} > bound {bound:.4g} (max|ref| {np.max(np.abs(ref)):.4g})"
    return err, bound
