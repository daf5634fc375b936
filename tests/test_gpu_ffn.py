"""SwiGLU block and MoE layer against the oracle.  Stage-wise protocol for the second mask: z on the GPU is
fp32 (expf) and the oracle's is binary64, so the two z can differ in the last bit; the GPU returns z_out, the
oracle recomputes the second mask from exactly those values (must match bit for bit) and the down projection
is compared both teacher-forced and end to end."""
import numpy as np
import pytest
import torch

import oracle
import scap_inputs as si
from scap_testlib import REL_L2_TOL, dev, f32, rel_l2_rows, workspace

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    import paper_2412_07174_b200 as scap
    scap.lib()
    return scap


def calibrate_glu(g, s1, s2, nbins=64, centre2=True):
    """Oracle-side calibration of both stages (stage 2 on the oracle's own z of the calibration tokens)."""
    dt = g["dt"]
    hc = si.to_f32(g["h_calib"], dt)
    m1, tau1 = oracle.calibrate(hc, s1, nbins)
    b1 = oracle.fold_bias(g["Wgu"], dt, m1, None)
    zc = oracle.glu_stage1_batch(hc, g["Wgu"], dt, m1, tau1, b1.astype(np.float32))
    m2, tau2 = oracle.calibrate(zc, s2, nbins if centre2 else 0)
    b2 = oracle.fold_bias(g["Wd"], dt, m2, None)
    return dict(m1=m1, tau1=tau1, b1=b1.astype(np.float32), m2=m2, tau2=tau2, b2=b2.astype(np.float32))


def run_glu(S, g, c, B=None):
    dt = g["dt"]
    h = dev(g["h"] if B is None else g["h"][:B], dt)
    Wgu, Wd = dev(g["Wgu"], dt), dev(g["Wd"], dt)
    B, D = h.shape
    F = g["F"]
    ws = workspace(S.scap_glu_workspace(B, D, F))
    yg, zg = workspace(B * D * 4), workspace(B * F * 4)
    y, z = yg.view(torch.float32, (B, D)), zg.view(torch.float32, (B, F))
    idx1 = torch.full((D,), -1, dtype=torch.int32, device="cuda")
    idx2 = torch.full((F,), -1, dtype=torch.int32, device="cuda")
    n1 = torch.zeros(1, dtype=torch.int32, device="cuda")
    n2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    S.scap_glu_ffn(h, Wgu, Wd, f32(c["m1"]), f32([c["tau1"]]), f32(c["b1"]), f32(c["m2"]), f32([c["tau2"]]), f32(c["b2"]),
                   y, ws.payload, z_out=z, idx1_out=idx1, nnz1_out=n1, idx2_out=idx2, nnz2_out=n2)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact() and zg.intact()
    return (y.cpu().numpy().copy(), z.cpu().numpy().copy(), idx1[: int(n1)].cpu().numpy().astype(np.uint32),
            idx2[: int(n2)].cpu().numpy().astype(np.uint32))


def check_glu(S, g, c, B=None):
    dt = g["dt"]
    hf = si.to_f32(g["h"] if B is None else g["h"][:B], dt)
    y, z, idx1, idx2 = run_glu(S, g, c, B)
    # stage 1 mask: bit-exact
    assert np.array_equal(idx1, oracle.mask(hf, c["m1"], c["tau1"])[2])
    # full oracle
    y64, z_o = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, c["m1"], c["tau1"], c["b1"], c["m2"], c["tau2"], c["b2"])
    assert rel_l2_rows(z, z_o.astype(np.float64)) <= 1e-5
    # stage 2 mask, recomputed by the oracle from the GPU's z: bit-exact
    keep2, _, idx2_o = oracle.mask(z, c["m2"], c["tau2"])
    assert np.array_equal(idx2, idx2_o)
    # teacher-forced down projection
    y_tf, _ = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, c["m1"], c["tau1"], c["b1"], c["m2"], c["tau2"], c["b2"], z_in=z)
    assert rel_l2_rows(y, y_tf) <= REL_L2_TOL
    # end to end; second-mask disagreements may only come from values within rounding of the threshold
    assert rel_l2_rows(y, y64) <= REL_L2_TOL
    keep2_o = oracle.mask(z_o, c["m2"], c["tau2"])[0]
    flips = keep2 != keep2_o
    if flips.any():
        dz = np.abs(z_o - c["m2"][None, :])
        assert np.all(np.abs(dz[flips] - c["tau2"]) <= 1e-5 * np.maximum(c["tau2"], dz[flips]))
    return keep2.mean()


@pytest.mark.parametrize("D,F,B", [(256, 512, 1), (200, 264, 3), (304, 520, 4), (512, 1000, 8), (64, 8, 2), (1024, 776, 16)])
def test_glu_small_shapes(S, D, F, B):
    g = si.glu_block(2, D, F, si.BF16, 64, B)
    c = calibrate_glu(g, 0.4, 0.7)
    kept2 = check_glu(S, g, c)
    assert kept2 < 0.9


@pytest.mark.parametrize("split", [3, 5, 6, 7])
@pytest.mark.parametrize("B", [1, 5])
def test_glu_cluster_sizes_that_do_not_divide_the_tile(S, split, B):
    g = si.glu_block(2, 520, 1000, si.BF16, 64, B)
    c = calibrate_glu(g, 0.4, 0.7)
    try:
        S.scap_tune("split_k", split)
        check_glu(S, g, c)
    finally:
        S.scap_tune("split_k", 0)


@pytest.mark.parametrize("D,F,B", [(520, 1000, 3), (1024, 776, 8), (2048, 520, 16)])
def test_glu_on_the_tcgen05_kernel(S, D, F, B):
    g = si.glu_block(2, D, F, si.BF16, 64, B)
    c = calibrate_glu(g, 0.4, 0.7)
    try:
        S.scap_tune("tcgen05", 2)
        S.scap_tune("dense_stream", 0)
        check_glu(S, g, c)
        S.scap_device_status()
    finally:
        S.scap_tune("tcgen05", 1)
        S.scap_tune("dense_stream", 1)


@pytest.mark.parametrize("D,F,B", [(520, 1000, 3), (1024, 776, 8), (2048, 520, 16), (200, 264, 5), (4096, 1376, 12)])
def test_glu_on_the_dense_stream_kernel(S, D, F, B):
    """Both stages on the TMA dense-stream kernel: packed gate|up boxes in the first, fp32 z as the input of the second."""
    g = si.glu_block(2, D, F, si.BF16, 64, B)
    c = calibrate_glu(g, 0.4, 0.7)
    try:
        S.scap_tune("dense_stream", 2)
        check_glu(S, g, c)
        S.scap_device_status()
    finally:
        S.scap_tune("dense_stream", 1)


def test_glu_fp16_and_no_centring(S):
    g = si.glu_block(2, 256, 520, si.F16, 64, 2)
    c = calibrate_glu(g, 0.3, 0.6, centre2=False)
    check_glu(S, g, c)


def test_glu_tau_zero_is_dense_swiglu(S):
    g = si.glu_block(2, 256, 264, si.BF16, 8, 2)
    D, F = 256, 264
    c = dict(m1=np.zeros(D, np.float32), tau1=0.0, b1=np.zeros(2 * F, np.float32), m2=np.zeros(F, np.float32), tau2=0.0,
             b2=np.zeros(D, np.float32))
    y, z, idx1, idx2 = run_glu(S, g, c)
    assert idx1.size == D and idx2.size == F
    hf = si.to_f32(g["h"], si.BF16).astype(np.float64)
    gu = hf @ si.to_f32(g["Wgu"], si.BF16).astype(np.float64)
    zz = gu[:, F:] * (gu[:, :F] / (1 + np.exp(-gu[:, :F])))
    assert rel_l2_rows(y, zz @ si.to_f32(g["Wd"], si.BF16).astype(np.float64)) <= REL_L2_TOL


def test_glu_is_deterministic(S):
    g = si.glu_block(2, 512, 776, si.BF16, 64, 4)
    c = calibrate_glu(g, 0.4, 0.7)
    a = run_glu(S, g, c)
    b = run_glu(S, g, c)
    assert all(np.array_equal(u, v) for u, v in zip(a, b))


# ---------------------------------------------------------------- MoE

def build_moe(D, F, E, B, T=64, s1=0.4, s2=0.6, nbins=64):
    mo = si.moe_layer(3, D, F, E, si.BF16, T, B)
    for p in mo["experts"]:
        g = dict(dt=si.BF16, h_calib=p["h_calib"], Wgu=p["Wgu"], Wd=p["Wd"])
        c = calibrate_glu(g, s1, s2, nbins)
        p.update(m1=c["m1"], tau1=c["tau1"], bgu_fused=c["b1"], m2=c["m2"], tau2=c["tau2"], bd_fused=c["b2"])
    return mo


def run_moe(S, mo, top_k=2):
    dt = mo["dt"]
    h = dev(mo["h"], dt)
    B, D = h.shape
    F, E = mo["F"], mo["E"]
    keep_alive = []
    experts = []
    for p in mo["experts"]:
        t = dict(Wgu=dev(p["Wgu"], dt), Wd=dev(p["Wd"], dt), m1=f32(p["m1"]), tau1=f32([p["tau1"]]),
                 bgu_fused=f32(p["bgu_fused"]), m2=f32(p["m2"]), tau2=f32([p["tau2"]]), bd_fused=f32(p["bd_fused"]))
        experts.append(t)
        keep_alive.append(t)
    ws = workspace(S.scap_moe_workspace(B, D, F, E, top_k))
    yg = workspace(B * D * 4)
    y = yg.view(torch.float32, (B, D))
    ex = torch.full((B, top_k), -1, dtype=torch.int32, device="cuda")
    w = torch.zeros((B, top_k), dtype=torch.float32, device="cuda")
    S.scap_moe_ffn(h, f32(mo["logits"]), experts, top_k, y, ws.payload, expert_out=ex, weight_out=w)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    return y.cpu().numpy().copy(), ex.cpu().numpy(), w.cpu().numpy()


@pytest.mark.parametrize("D,F,E,B,top_k", [(256, 520, 8, 4, 2), (128, 264, 4, 1, 2), (256, 256, 3, 5, 1), (64, 72, 8, 16, 2)])
def test_moe_small(S, D, F, E, B, top_k):
    mo = build_moe(D, F, E, B)
    y, ex, w = run_moe(S, mo, top_k)
    y64, ex_o, w_o = oracle.moe_ffn(si.to_f32(mo["h"], mo["dt"]), mo["logits"], mo["experts"], mo["dt"], top_k)
    assert np.array_equal(ex, ex_o)
    assert np.allclose(w, w_o, rtol=1e-6, atol=0)
    assert rel_l2_rows(y, y64) <= REL_L2_TOL


# ---------------------------------------------------------------- non-GLU FFN (up -> exact GELU -> centred sparse down)

def gelu_block(D, F, B, dt=si.BF16, T=64):
    """A [D, F] up weight (the up half of the packed recipe), the down weight and inputs of the SwiGLU recipe."""
    g = si.glu_block(2, D, F, dt, T, B)
    g["Wu"] = np.ascontiguousarray(g["Wgu"][:, F:])
    return g


def calibrate_gelu(g, s1, s2, nbins=64):
    dt = g["dt"]
    hc = si.to_f32(g["h_calib"], dt)
    m1, tau1 = oracle.calibrate(hc, s1, nbins)
    b1 = oracle.fold_bias(g["Wu"], dt, m1, None).astype(np.float32)
    _, zc = oracle.gelu_ffn(hc, g["Wu"], g["Wd"], dt, m1, tau1, b1, None, 0.0, None)
    m2, tau2 = oracle.calibrate(zc, s2, nbins)
    b2 = oracle.fold_bias(g["Wd"], dt, m2, None).astype(np.float32)
    return dict(m1=m1, tau1=tau1, b1=b1, m2=m2, tau2=tau2, b2=b2)


def check_gelu(S, g, c):
    dt = g["dt"]
    hf = si.to_f32(g["h"], dt)
    h, Wu, Wd = dev(g["h"], dt), dev(g["Wu"], dt), dev(g["Wd"], dt)
    B, D = h.shape
    F = g["F"]
    ws = workspace(S.scap_gelu_ffn_workspace(B, D, F))
    yg, zg = workspace(B * D * 4), workspace(B * F * 4)
    y, z = yg.view(torch.float32, (B, D)), zg.view(torch.float32, (B, F))
    idx1 = torch.full((D,), -1, dtype=torch.int32, device="cuda")
    idx2 = torch.full((F,), -1, dtype=torch.int32, device="cuda")
    n1 = torch.zeros(1, dtype=torch.int32, device="cuda")
    n2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    S.scap_gelu_ffn(h, Wu, Wd, f32(c["m1"]), f32([c["tau1"]]), f32(c["b1"]), f32(c["m2"]), f32([c["tau2"]]), f32(c["b2"]),
                    y, ws.payload, z_out=z, idx1_out=idx1, nnz1_out=n1, idx2_out=idx2, nnz2_out=n2)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact() and zg.intact()
    y, z = y.cpu().numpy().copy(), z.cpu().numpy().copy()
    idx1, idx2 = idx1[: int(n1)].cpu().numpy().astype(np.uint32), idx2[: int(n2)].cpu().numpy().astype(np.uint32)
    assert np.array_equal(idx1, oracle.mask(hf, c["m1"], c["tau1"])[2])                      # stage-1 mask: bit-exact
    y64, z_o = oracle.gelu_ffn(hf, g["Wu"], g["Wd"], dt, c["m1"], c["tau1"], c["b1"], c["m2"], c["tau2"], c["b2"])
    assert np.max(np.abs(z - z_o)) <= 2e-6 * max(1.0, float(np.max(np.abs(z_o))))          # erff vs erf, fp32 accumulation
    keep2, _, idx2_o = oracle.mask(z, c["m2"], c["tau2"])                                    # stage-2 mask from the GPU's z
    assert np.array_equal(idx2, idx2_o)
    y_tf, _ = oracle.gelu_ffn(hf, g["Wu"], g["Wd"], dt, c["m1"], c["tau1"], c["b1"], c["m2"], c["tau2"], c["b2"], z_in=z)
    assert rel_l2_rows(y, y_tf) <= REL_L2_TOL
    assert rel_l2_rows(y, y64) <= REL_L2_TOL
    keep2_o = oracle.mask(z_o, c["m2"], c["tau2"])[0]
    flips = keep2 != keep2_o
    if flips.any():
        dz = np.abs(z_o - c["m2"][None, :])
        assert np.all(np.abs(dz[flips] - c["tau2"]) <= 1e-5 * np.maximum(c["tau2"], dz[flips]))
    return keep2.mean()


@pytest.mark.parametrize("tc_mode", [1, 2])
@pytest.mark.parametrize("D,F,B", [(256, 512, 1), (200, 264, 3), (512, 1000, 8), (64, 8, 2), (1024, 776, 16)])
def test_gelu_ffn_small_shapes(S, D, F, B, tc_mode):
    g = gelu_block(D, F, B)
    c = calibrate_gelu(g, 0.3, 0.5)
    try:
        S.scap_tune("tcgen05", tc_mode)
        S.scap_tune("dense_stream", 0 if tc_mode == 2 else 1)   # 2: the gather tcgen05 kernel, 1: the default routes
        kept2 = check_gelu(S, g, c)
    finally:
        S.scap_tune("tcgen05", 1)
        S.scap_tune("dense_stream", 1)
    assert kept2 < 0.95


def test_gelu_ffn_dense_up_projection_and_fp16(S):
    g = gelu_block(264, 520, 4, dt=si.F16)
    c = calibrate_gelu(g, 0.3, 0.5)
    c["tau1"] = np.float32(0.0)                                   # every input channel of the up projection kept
    check_gelu(S, g, c)
