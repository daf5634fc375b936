"""Parity at the full sizes of the five workload descriptions, in the launch configuration bench.py times
(automatic tile width / cluster size, programmatic dependent launch on).  The oracle is fast enough to compute
every output element at these sizes, so the comparison is element by element, not sampled."""
import numpy as np
import pytest
import torch

import oracle
import scap_inputs as si
from scap_testlib import REL_L2_TOL, dev, f32, rel_l2_rows, workspace
from test_gpu_ffn import calibrate_glu, check_glu, run_moe

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    import paper_2412_07174_b200 as scap
    scap.lib()
    return scap


def gpu_calibrate_and_fold(S, xc_bits, W_bits, b_bits, dt, s, nbins=2048):
    """Product-path calibration: m, tau from scap_calibrate, b_fused from scap_fold_bias (device tensors)."""
    xc, W = dev(xc_bits, dt), dev(W_bits, dt)
    T, K = xc.shape
    N = W.shape[1]
    m = torch.empty(K, dtype=torch.float32, device="cuda")
    tau = torch.empty(1, dtype=torch.float32, device="cuda")
    bf = torch.empty(N, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(S.scap_calibrate_workspace(T, K, nbins), S.scap_fold_bias_workspace(K, N)), dtype=torch.uint8,
                     device="cuda")
    S.scap_calibrate(xc, s, nbins, m, tau, ws)
    S.scap_fold_bias(W, m, None if b_bits is None else dev(b_bits, dt), bf, ws)
    torch.cuda.synchronize()
    return W, m, tau, bf


def sparse_parity(S, d, W, m, tau, bf, x_bits, m_o, tau_o, bf64):
    dt = d["dt"]
    x = dev(x_bits, dt)
    B, K = x.shape
    N = W.shape[1]
    ws = workspace(S.scap_fc_workspace(B, K, N))
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    idx = torch.empty(K, dtype=torch.int32, device="cuda")
    nnz = torch.zeros(1, dtype=torch.int32, device="cuda")
    S.scap_sparse_fc(x, W, m, tau, bf, y, ws.payload, idx_out=idx, nnz_out=nnz)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    xf = si.to_f32(x_bits, dt)
    y64 = oracle.sparse_fc(xf, d["W"], dt, m_o, tau_o, None, threads=8) + bf64[None, :]
    idx_o = oracle.mask(xf, m_o, tau_o)[2]
    n = int(nnz.item())
    assert n == idx_o.size and np.array_equal(idx[:n].cpu().numpy().astype(np.uint32), idx_o)
    assert rel_l2_rows(y.cpu().numpy(), y64) <= REL_L2_TOL
    return n / K


@pytest.mark.parametrize("s", [0.5, 0.65, 0.8])
def test_config1_llama_down_projection(S, s):
    d = si.config1(B=2)
    dt = d["dt"]
    xcf = si.to_f32(d["x_calib"], dt)
    m_o, tau_o = oracle.calibrate(xcf, s, 2048)
    bf64 = oracle.fold_bias(d["W"], dt, m_o, None)
    W, m, tau, bf = gpu_calibrate_and_fold(S, d["x_calib"], d["W"], None, dt, s)
    assert np.array_equal(m.cpu().numpy(), m_o) and float(tau.item()) == float(tau_o)
    got = bf.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - bf64) / np.linalg.norm(bf64) <= 1e-6
    for b in range(2):  # batch 1, two different tokens
        kept = sparse_parity(S, d, W, m, tau, bf, d["x"][b:b + 1], m_o, tau_o, bf64)
        assert abs((1 - kept) - s) < 0.03     # observed sparsity tracks the target (Appendix A)


@pytest.fixture(scope="module")
def config2_calibrated():
    g = si.config2(B=8)
    return g, calibrate_glu(g, 0.4, 0.7, nbins=2048)   # 1024 calibration tokens through the oracle: done once


@pytest.mark.parametrize("B", [1, 4, 8])
def test_config2_llama_swiglu_block(S, config2_calibrated, B):
    g, c = config2_calibrated
    kept2 = check_glu(S, g, c, B=B)
    assert kept2 < 0.6


def test_config3_mixtral_moe_layer(S):
    D, F, E, B = 4096, 14336, 8, 4
    mo = si.moe_layer(3, D, F, E, si.BF16, 2048, B)
    for p in mo["experts"]:
        hc = si.to_f32(p["h_calib"], si.BF16)
        m1, tau1 = oracle.calibrate(hc, 0.4, 2048)
        b1 = oracle.fold_bias(p["Wgu"], si.BF16, m1, None).astype(np.float32)
        # stage 2 is calibrated on the oracle's z of all 2048 calibration tokens of this expert, as the workload
        # description says (in slabs of 512 rows, to bound the host memory of the float64 product)
        zc = np.concatenate([oracle.glu_stage1_batch(hc[t:t + 512], p["Wgu"], si.BF16, m1, tau1, b1) for t in range(0, hc.shape[0], 512)])
        assert zc.shape == (2048, F)
        m2, tau2 = oracle.calibrate(zc, 0.6, 2048)
        b2 = oracle.fold_bias(p["Wd"], si.BF16, m2, None).astype(np.float32)
        p.update(m1=m1, tau1=tau1, bgu_fused=b1, m2=m2, tau2=tau2, bd_fused=b2)
    hf = si.to_f32(mo["h"], si.BF16)
    for nb in (1, 2, 3, 4):
        sub = dict(mo, h=mo["h"][:nb], logits=mo["logits"][:nb])
        y, ex, w = run_moe(S, sub, 2)
        y64, ex_o, w_o = oracle.moe_ffn(hf[:nb], sub["logits"], mo["experts"], si.BF16, 2)
        assert np.array_equal(ex, ex_o)
        assert np.allclose(w, w_o, rtol=1e-6, atol=0)
        assert rel_l2_rows(y, y64) <= REL_L2_TOL


@pytest.mark.parametrize("K,N", [(4096, 4096), (4096, 11008), (11008, 4096), (14336, 4096)])
def test_config4_sweep_points(S, K, N):
    d = si.config4_fc(K, N, 16, T_calib=256)
    dt = d["dt"]
    xcf = si.to_f32(d["x_calib"], dt)
    m_o = oracle.mode(xcf, 2048)
    bf64 = oracle.fold_bias(d["W"], dt, m_o, None)
    W = dev(d["W"], dt)
    m, bf = f32(m_o), f32(bf64)
    for s, B in [(0.0, 1), (0.6, 1), (0.9, 1), (0.6, 2), (0.6, 4), (0.8, 4), (0.5, 8), (0.25, 16), (0.9, 16)]:
        tau_o = oracle.tau(xcf, m_o, s)
        sparse_parity(S, d, W, m, f32([tau_o]), bf, d["x"][:B], m_o, tau_o, bf64)
    # dense baseline on the same layer
    x = dev(d["x"][:4], dt)
    ws = workspace(S.scap_fc_workspace(4, K, N))
    y = torch.empty((4, N), dtype=torch.float32, device="cuda")
    S.scap_dense_fc(x, W, None, y, ws.payload)
    torch.cuda.synchronize()
    y64 = oracle.dense_fc(si.to_f32(d["x"][:4], dt), d["W"], dt, None)
    assert rel_l2_rows(y.cpu().numpy(), y64) <= REL_L2_TOL


@pytest.mark.parametrize("B", [1, 4])
def test_fused_qkv_projection_shares_one_mask(S, B):
    """Q, K and V read the same input, so the fused projection is one sparse FC on the packed [D, 3D] weight with one
    kept-channel list (Section 1 of the paper: projections that share their input share its mask)."""
    D = 4096
    d = si.config4_fc(D, 3 * D, 4, T_calib=256)
    dt = d["dt"]
    xcf = si.to_f32(d["x_calib"], dt)
    m_o, tau_o = oracle.calibrate(xcf, 0.5, 2048)
    bf64 = oracle.fold_bias(d["W"], dt, m_o, None)
    sparse_parity(S, d, dev(d["W"], dt), f32(m_o), f32([tau_o]), f32(bf64), d["x"][:B], m_o, tau_o, bf64)
