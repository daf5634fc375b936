"""scap_glu_ffn_static: the SwiGLU block for callers that are not allowed to allocate device memory (a server
whose HBM is fully committed to its own pools, a plug-in inside another framework's budget, a latency-critical
loop that cannot afford cudaMalloc's device synchronisation).  Its scratch is a fixed array inside the library.

The test calls it through the C ABI twice in a row with different inputs and checks each result against the
ordinary scap_glu_ffn (caller workspace) on the same inputs - bit for bit, since both run the same kernels - and
against the CPU oracle within the tolerance the other GPU tests use; it checks that the calls leave the amount of
free device memory unchanged, and that a shape beyond the built-in capacity is refused before anything is launched.  This file sorts
last on purpose, so a run that stops at the first failure has already run every other test; it passes both on
its own in a fresh process and after the other tests."""
import numpy as np
import pytest
import torch

import oracle
import scap_inputs as si
from scap_testlib import REL_L2_TOL, dev, f32, rel_l2_rows, workspace

pytestmark = pytest.mark.gpu


def test_static_scratch_swiglu_matches_workspace_version_twice():
    import paper_2412_07174_b200 as scap
    scap.lib()
    D, F, B = 512, 1032, 4
    cap = scap.scap_glu_static_capacity()
    assert scap.scap_glu_workspace(B, D, F) <= cap
    g = si.glu_block(2, D, F, si.BF16, 8, 2 * B)
    dt = si.BF16
    Wgu, Wd = dev(g["Wgu"], dt), dev(g["Wd"], dt)
    m1 = f32(np.linspace(-0.05, 0.05, D))
    m2 = f32(np.full(F, 0.001))
    tau1, tau2 = f32([0.5]), f32([0.02])
    b1 = f32(np.linspace(-0.01, 0.01, 2 * F))
    b2 = f32(np.linspace(0.02, -0.02, D))
    ws = workspace(scap.scap_glu_workspace(B, D, F))
    m1_o, m2_o = m1.cpu().numpy(), m2.cpu().numpy()
    b1_o, b2_o = b1.cpu().numpy(), b2.cpu().numpy()
    warm = torch.empty((B, D), dtype=torch.float32, device="cuda")
    scap.scap_glu_ffn_static(dev(g["h"][:B], dt), Wgu, Wd, m1, tau1, b1, m2, tau2, b2, warm)  # first call: address look-up
    torch.cuda.synchronize()
    for call in range(2):                       # two calls in a row, different activations, one shared scratch
        h = dev(g["h"][call * B:(call + 1) * B], dt)
        y_ref = torch.empty((B, D), dtype=torch.float32, device="cuda")
        z_ref = torch.empty((B, F), dtype=torch.float32, device="cuda")
        scap.scap_glu_ffn(h, Wgu, Wd, m1, tau1, b1, m2, tau2, b2, y_ref, ws.payload, z_out=z_ref)
        yg = workspace(B * D * 4)
        y = yg.view(torch.float32, (B, D))
        z = torch.empty((B, F), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        scap.scap_glu_ffn_static(h, Wgu, Wd, m1, tau1, b1, m2, tau2, b2, y, z_out=z)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before   # the call allocated no device memory
        assert yg.intact() and ws.intact()
        assert float(y_ref.abs().max()) > 0
        assert torch.equal(z, z_ref) and torch.equal(y, y_ref)   # same kernels, same inputs: the same bits
        # and against the oracle: its own z for the stage-1 check, the GPU's z fed back for the final product
        hf = si.to_f32(g["h"][call * B:(call + 1) * B], dt)
        y64, z_o = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, m1_o, 0.5, b1_o, m2_o, 0.02, b2_o)
        assert rel_l2_rows(z.cpu().numpy(), z_o.astype(np.float64)) <= 1e-5
        y64_fed, _ = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, m1_o, 0.5, b1_o, m2_o, 0.02, b2_o, z_in=z.cpu().numpy())
        assert rel_l2_rows(y.cpu().numpy(), y64_fed) <= REL_L2_TOL
        assert rel_l2_rows(y.cpu().numpy(), y64) <= REL_L2_TOL


def test_static_scratch_rejects_shapes_beyond_its_capacity():
    import paper_2412_07174_b200 as scap
    L = scap.lib()
    cap = scap.scap_glu_static_capacity()
    B, D, F = 16, 64, 40000
    assert scap.scap_glu_workspace(B, D, F) > cap
    P = 0x10000  # never dereferenced: the size check comes first
    assert L.scap_glu_ffn_static(P, P, P, None, P, None, None, P, None, P, B, D, F, 1, None, None) == 5  # SCAP_ERR_WORKSPACE
    assert L.scap_glu_ffn_static(P, P, P, None, P, None, None, P, None, P, 0, D, 64, 1, None, None) == 2  # SCAP_ERR_SHAPE
