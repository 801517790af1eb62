"""The allocation-free forward entry point (for callers that cannot allocate device memory when
they run the operator) against the regular forward, through the C ABI, twice in a row.  This
file sorts last so that a run stopping at the first failure has already run every other test."""
import numpy as np
import pytest

from workloads import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_forward_matches_workspace_forward():
    import torch
    import paper_2607_18074_b200 as sb
    from gpu_util import FWD_TOL, Case, rel_err

    # cfg5 irreps: 920 KiB of state per node, so the 32 MiB array forces several node chunks
    for w in (synth.scaled(synth.config("cfg2"), 300), synth.scaled(synth.config("cfg5"), 70)):
        c = Case(w)
        ref = c.fwd()                                   # existing entry point, caller's workspace
        before = torch.cuda.memory_allocated()
        for _ in range(2):                              # second call sees the first call's leftovers
            y = torch.full((c.N, c.plan.info.C_y), float("nan"), dtype=torch.float32, device="cuda:0")
            sb.conv_fwd_static(c.plan, c.graph, c.x, c.Y, c.phi, c.R, y)
            assert sb.static_last_status() == 0         # no bounded wait gave up, no id out of range
            got = y.cpu().numpy()
            assert np.isfinite(got).all()
            assert rel_err(got, ref) <= FWD_TOL
            del y
        assert torch.cuda.memory_allocated() == before


def test_static_scratch_rejects_oversized_contracts():
    import ctypes
    import torch
    import paper_2607_18074_b200 as sb
    # one node's state alone (K * F floats) exceeds the array
    ir = [(2048, 0, 1), (2048, 1, -1)]
    plan = sb.Plan(ir, ir, 1, 16)
    need = 256 + 4 * 16 * plan.info.N_w + 4 * plan.info.state_floats_fwd
    assert need > sb.static_scratch_bytes()
    # real (tiny) device buffers: the size check refuses the call before anything is launched, and if it ever
    # did not, the kernels would read valid memory
    rp = torch.tensor([0, 1], dtype=torch.int64, device="cuda:0")
    col = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    buf = torch.zeros(64, dtype=torch.float32, device="cuda:0")
    b = ctypes.c_void_p(buf.data_ptr())
    rc = sb.lib().sobek_conv_fwd_static(plan.handle, ctypes.byref(sb.make_graph(rp, col)), b, b, b, b, b, None)
    assert rc == -3
