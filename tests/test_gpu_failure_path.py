"""The failure path on the device: a bounded wait that runs out.

The paper's run-time failure is a wait that never ends (subgraphs that depend on each other deadlock: Section II, last
paragraph; Section IV, "Acyclic Partitioning"). On the device its counterpart is a wait on a signal that never comes.
Every such wait of the library is bounded. These tests make one run out on a tiny problem through the library's test
hook: the producer of one mbarrier skips its arrival and the wait budget is set to 2 ms. Nothing faults, traps or spins
without a limit; the kernel runs to its end, frees its tensor memory, the handle reports AGO_ERR_TIMEOUT with the wait
site, and the next ordinary run on the same handle matches the oracle."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2212_01005_b200 import workloads as WL
from helpers import assert_close, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,site", [("fused", 0x104), ("per_mini_subgraph", 0x503)])
def test_bounded_wait_runs_out_and_the_handle_recovers(ago, mode, site):
    import torch
    wl = WL.get("mbv2_14")
    data = WL.generate(wl)
    ref = O.run_chain(wl.ops, data["inputs"], data["weights"])
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode=mode)
    ins, ws = to_device(wl, data)

    # an ordinary run first: the status block exists and reads OK
    out = sg.run(ins, ws)
    assert sg.status() == ago.AGO_OK, ago.ago_last_error()
    assert_close(out.float().cpu().numpy().astype(np.float64), ref, what=f"{mode} before the injected timeout")

    assert ago.ago_subgraph_debug(sg._h, ago.AGO_DEBUG_WAIT_BUDGET_US, 2000) == ago.AGO_OK
    assert ago.ago_subgraph_debug(sg._h, ago.AGO_DEBUG_SKIP_SIGNAL, site) == ago.AGO_OK
    sg.run(ins, ws)
    torch.cuda.synchronize()                      # the kernel came back by itself
    st = sg.status()
    code, msg = ago.ago_last_error()
    assert st == ago.AGO_ERR_TIMEOUT, (st, msg)
    assert f"0x{site:x}" in msg, msg
    assert sg.status() == ago.AGO_OK              # the word was cleared by the read

    # hook off, default budget: the same handle, the same context, a correct result
    assert ago.ago_subgraph_debug(sg._h, ago.AGO_DEBUG_SKIP_SIGNAL, 0) == ago.AGO_OK
    assert ago.ago_subgraph_debug(sg._h, ago.AGO_DEBUG_WAIT_BUDGET_US, 0) == ago.AGO_OK
    out = sg.run(ins, ws)
    torch.cuda.synchronize()
    assert sg.status() == ago.AGO_OK, ago.ago_last_error()
    assert_close(out.float().cpu().numpy().astype(np.float64), ref, what=f"{mode} after the injected timeout")
    sg.close()


def test_debug_hook_rejects_bad_arguments(ago):
    wl = WL.get("mbv2_14")
    sg = ago.Subgraph(wl.ops, wl.input_shapes, mode="fused")
    assert ago.ago_subgraph_debug(sg._h, 99, 0) == ago.AGO_ERR_INVALID_ARG
    assert ago.ago_subgraph_debug(sg._h, ago.AGO_DEBUG_WAIT_BUDGET_US, -1) == ago.AGO_ERR_INVALID_ARG
    assert ago.ago_subgraph_debug(None, ago.AGO_DEBUG_WAIT_BUDGET_US, 1) == ago.AGO_ERR_INVALID_ARG
    sg.close()
