"""Sparse FC on 8-bit weights (per-input-channel scales) against the oracle: kept list bit-exact, y within 2e-3 rel-L2."""
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


def case(K, N, B, dt):
    d = si.laplace_fc(4, K, N, dt, 16, B)
    q, scale = si.quantise_q8(d["W"], dt)
    d["Wq"], d["wscale"] = q, scale
    return d


def run_q8(S, d, m, tau, bf, want_idx=True):
    dt = d["dt"]
    x = dev(d["x"], dt)
    Wq = torch.from_numpy(d["Wq"]).cuda()
    B, K = x.shape
    N = Wq.shape[1]
    ws = workspace(S.scap_fc_workspace(B, K, N))
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    idx = torch.full((K,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    nnz = torch.full((1,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    S.scap_sparse_fc_q8(x, Wq, f32(d["wscale"]), None if m is None else f32(m), f32([tau]), None if bf is None else f32(bf), y,
                        ws.payload, idx_out=idx, nnz_out=nnz)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    gi = idx[: int(nnz.item())].cpu().numpy().astype(np.uint32) if want_idx else None
    return y.cpu().numpy().copy(), gi


@pytest.mark.parametrize("K,N,B,dt", [
    (1024, 1024, 1, si.F16), (1500, 528, 1, si.BF16), (1500, 528, 2, si.BF16), (4100, 272, 2, si.F16), (96, 16, 1, si.BF16),
    (11008, 4096, 1, si.BF16), (11008, 4096, 2, si.BF16), (14336, 512, 1, si.BF16), (14336, 512, 2, si.F16),
])
def test_q8_sparse_fc_matches_the_oracle(S, K, N, B, dt):
    d = case(K, N, B, dt)
    xf = si.to_f32(d["x"], dt)
    m = d["m_true"]
    bf64 = oracle.fold_bias_q8(d["Wq"], d["wscale"], m, None)
    for tau in (0.25, 0.0):
        y64 = oracle.sparse_fc_q8(xf, d["Wq"], d["wscale"], m, tau, bf64.astype(np.float32))
        y, gidx = run_q8(S, d, m, tau, bf64.astype(np.float32))
        assert np.array_equal(gidx, oracle.mask(xf, m, tau)[2])
        assert rel_l2_rows(y, y64) <= REL_L2_TOL


def test_q8_batches_beyond_two_rows_and_the_dense_and_folding_calls(S):
    d = case(2048, 544, 5, si.BF16)
    xf = si.to_f32(d["x"], si.BF16)
    m = d["m_true"]
    Wq, sc = torch.from_numpy(d["Wq"]).cuda(), f32(d["wscale"])
    ws = workspace(S.scap_fc_workspace(5, 2048, 544))
    # folding on the device against the oracle
    bfg = torch.empty(544, dtype=torch.float32, device="cuda")
    bias = np.linspace(-1, 1, 544).astype(np.float32)
    S.scap_fold_bias_q8(Wq, sc, f32(m), f32(bias), bfg, ws.payload)
    torch.cuda.synchronize()
    bf64 = oracle.fold_bias_q8(d["Wq"], d["wscale"], m, bias)
    assert rel_l2_rows(bfg.cpu().numpy(), bf64) <= 1e-6
    # five rows (two + two + one launches): every row equals its own batch-1 result definition
    y64 = oracle.sparse_fc_q8(xf, d["Wq"], d["wscale"], m, 0.3, bf64.astype(np.float32))
    y, _ = run_q8(S, d, m, 0.3, bf64.astype(np.float32), want_idx=False)
    assert rel_l2_rows(y, y64) <= REL_L2_TOL
    # dense call = tau 0 without centring
    yd = torch.empty((5, 544), dtype=torch.float32, device="cuda")
    S.scap_dense_fc_q8(dev(d["x"], si.BF16), Wq, sc, f32(bias), yd, ws.payload)
    torch.cuda.synchronize()
    assert rel_l2_rows(yd.cpu().numpy(), oracle.sparse_fc_q8(xf, d["Wq"], d["wscale"], None, 0.0, bias)) <= REL_L2_TOL
    assert ws.intact()


def test_q8_nothing_kept_returns_the_bias_and_rejects_bad_shapes(S):
    d = case(640, 272, 2, si.BF16)
    bf = np.linspace(-1, 1, 272).astype(np.float32)
    y, gidx = run_q8(S, d, d["m_true"], np.inf, bf)
    assert gidx.size == 0 and np.array_equal(y, np.tile(bf, (2, 1)))
    x = dev(d["x"], si.BF16)
    ws = workspace(S.scap_fc_workspace(2, 640, 272))
    yb = torch.empty((2, 264), dtype=torch.float32, device="cuda")
    with pytest.raises(S.ScapError):  # N not a multiple of 16
        S.scap_sparse_fc_q8(x, torch.zeros((640, 264), dtype=torch.int8, device="cuda"), f32(d["wscale"]), None, f32([0.1]), None, yb, ws.payload)
