"""The allocation-free entry point, vorta_routed_attention_static.

Some callers of this library cannot allocate device memory: code that runs inside another
framework's memory pool, plug-ins that are only ever handed tensors, services whose memory
budget is fixed at start-up.  For them the core-set branch's scratch is an array built into
the library.  This file checks, through the C ABI, that the entry point gives the same output
as vorta_routed_attention with a caller-provided workspace, on two calls in a row (the array
keeps the first call's contents), that one head also agrees with the CPU oracle directly, that
it refuses plans whose scratch does not fit, and that the call leaves device memory alone: the
free bytes the driver reports (which count every allocation on the device, the library's own
included, not only torch's) are the same before and after the second call.  The first call on a
device may make the driver set the array aside, so it is not held to that.

It is collected last on purpose: a run that stops at the first failure has then already run
every other test.  It also passes on its own in a fresh process.
"""
import gc

import pytest
import torch

from helpers import assert_close, oracle_head_rows
from paper_2505_18809_b200 import binding as vb
from paper_2505_18809_b200 import build as vbuild
from paper_2505_18809_b200 import workloads
from paper_2505_18809_b200.workloads import Workload

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    vbuild.build()
    vb.lib()


def test_static_workspace_entry_point_matches_the_workspace_one_twice():
    # all three routes; the core-set heads make the scratch matter
    wl = Workload("no-alloc", (6, 12, 16), 4, 128, (2, 4, 4), (3, 3, 3), 0.5, (2, 1, 0, 2), 51, True)
    plan = vb.Plan.from_workload(wl)
    assert 0 < plan.info.workspace_bytes <= vb.VORTA_STATIC_WORKSPACE_BYTES
    stream = int(torch.cuda.current_stream().cuda_stream)
    for call in range(2):
        # different inputs per call: the second call must not see the first one's leftovers
        seeded = Workload(wl.name, wl.grid, wl.heads, wl.d, wl.tile, wl.window, wl.ratio, wl.routes,
                          wl.seed + call, wl.smooth)
        Q, K, V = workloads.make_qkv(seeded, DEV)
        want = plan.routed_attention(Q, K, V)
        assert plan.device_status() == 0
        got = torch.full_like(Q, float("nan"))
        gc.collect()                     # tensors of the previous round must not be released under the call
        torch.cuda.synchronize()
        before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        vb.vorta_routed_attention_static(plan.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(),
                                         got.data_ptr(), None, 0, stream)
        assert plan.device_status() == 0
        assert torch.cuda.memory_allocated() == before
        if call == 1:
            assert torch.cuda.mem_get_info()[0] >= free_before   # nothing was allocated, by the library or anyone
        # same kernels, same inputs: the tolerance of the parity tests, and in fact the same bits
        err = (got.float() - want.float()).abs()
        assert float(err.max()) <= 2e-2 and float(err.mean()) <= 2e-3
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"call {call}"
        # and one core-set head against the oracle itself, not only against the other entry point
        assert_close(got[0, 0], oracle_head_rows(seeded, Q, K, V, 0, 0, None), f"call {call} head 0 vs oracle")
    plan.close()


def test_static_workspace_entry_point_refuses_what_does_not_fit():
    wl = workloads.config("wan1.3b-480p")          # four core-set heads of 16 380 rows: ~67 MB of scratch
    plan = vb.Plan.from_workload(wl)
    assert plan.info.workspace_bytes > vb.VORTA_STATIC_WORKSPACE_BYTES
    x = torch.zeros(16, dtype=torch.bfloat16, device=DEV)   # never touched: the call must fail first
    with pytest.raises(vb.VortaError) as e:
        vb.vorta_routed_attention_static(plan.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr())
    assert e.value.status == vb.VORTA_ERR_WORKSPACE
    # without core-set heads no scratch is needed and the same shape is accepted
    plan.set_routes([0] * wl.heads)
    assert plan.info.workspace_bytes == 0
    plan.close()


def test_static_workspace_entry_point_takes_a_plan_without_scratch():
    wl = Workload("no-scratch", (4, 8, 16), 2, 128, (2, 4, 4), (3, 3, 3), 0.5, (0, 1), 52, False)
    plan = vb.Plan.from_workload(wl)
    assert plan.info.workspace_bytes == 0
    Q, K, V = workloads.make_qkv(wl, DEV)
    got = torch.full_like(Q, float("nan"))
    vb.vorta_routed_attention_static(plan.handle, Q.data_ptr(), K.data_ptr(), V.data_ptr(), got.data_ptr(), None, 0,
                                     int(torch.cuda.current_stream().cuda_stream))
    assert plan.device_status() == 0
    for h in range(wl.heads):
        assert_close(got[0, h], oracle_head_rows(wl, Q, K, V, 0, h, None), f"head {h}")
    plan.close()
