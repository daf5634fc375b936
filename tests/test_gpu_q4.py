"""Sparse FC on group-wise 4-bit weights (two codes per byte; scale and zero point per group of input channels and output
column) against the oracle: kept list bit-exact, y within 2e-3 rel-L2 of the oracle's binary64 result on the same codes."""
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


def case(K, N, B, dt, group):
    d = si.laplace_fc(4, K, N, dt, 16, B)
    d["Wq"], d["scale"], d["zero"] = si.quantise_q4(d["W"], dt, group)
    d["group"] = group
    return d


def run_q4(S, d, m, tau, bf, want_idx=True):
    dt = d["dt"]
    x = dev(d["x"], dt)
    Wq, zero = torch.from_numpy(d["Wq"]).cuda(), torch.from_numpy(d["zero"]).cuda()
    B, K = x.shape
    N = Wq.shape[1] * 2
    ws = workspace(S.scap_fc_workspace(B, K, N))
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    idx = torch.full((K,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    nnz = torch.full((1,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    S.scap_sparse_fc_q4(x, Wq, f32(d["scale"]), zero, d["group"], None if m is None else f32(m), f32([tau]),
                        None if bf is None else f32(bf), y, ws.payload, idx_out=idx, nnz_out=nnz)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    gi = idx[: int(nnz.item())].cpu().numpy().astype(np.uint32) if want_idx else None
    return y.cpu().numpy().copy(), gi


@pytest.mark.parametrize("K,N,B,dt,group", [
    (1024, 1024, 1, si.F16, 128), (1500, 528, 1, si.BF16, 128), (1500, 528, 2, si.BF16, 64), (4100, 272, 2, si.F16, 32),
    (96, 16, 1, si.BF16, 32), (3000, 1040, 1, si.BF16, 256), (11008, 4096, 1, si.BF16, 128),
])
def test_q4_sparse_fc_matches_the_oracle(S, K, N, B, dt, group):
    d = case(K, N, B, dt, group)
    xf = si.to_f32(d["x"], dt)
    m = d["m_true"]
    bf64 = oracle.fold_bias_q4(d["Wq"], d["scale"], d["zero"], group, m, None)
    for tau in (0.25, 0.0):
        y64 = oracle.sparse_fc_q4(xf, d["Wq"], d["scale"], d["zero"], group, m, tau, bf64.astype(np.float32))
        y, gidx = run_q4(S, d, m, tau, bf64.astype(np.float32))
        assert np.array_equal(gidx, oracle.mask(xf, m, tau)[2])
        assert rel_l2_rows(y, y64) <= REL_L2_TOL


@pytest.mark.parametrize("split", [1, 3, 8])
def test_q4_cluster_sizes(S, split):
    d = case(2304, 784, 2, si.BF16, 128)     # 18 groups over 1, 3 or 8 ranks (some ranks get fewer, or none)
    xf = si.to_f32(d["x"], si.BF16)
    m = d["m_true"]
    try:
        S.scap_tune("split_k", split)
        y64 = oracle.sparse_fc_q4(xf, d["Wq"], d["scale"], d["zero"], 128, m, 0.2, None)
        y, gidx = run_q4(S, d, m, 0.2, None)
        assert np.array_equal(gidx, oracle.mask(xf, m, 0.2)[2])
        assert rel_l2_rows(y, y64) <= REL_L2_TOL
    finally:
        S.scap_tune("split_k", 0)


def test_q4_batches_beyond_two_rows_and_the_dense_and_folding_calls(S):
    d = case(2048, 544, 5, si.BF16, 128)
    xf = si.to_f32(d["x"], si.BF16)
    m = d["m_true"]
    Wq, zero, sc = torch.from_numpy(d["Wq"]).cuda(), torch.from_numpy(d["zero"]).cuda(), f32(d["scale"])
    ws = workspace(S.scap_fc_workspace(5, 2048, 544))
    bfg = torch.empty(544, dtype=torch.float32, device="cuda")
    bias = np.linspace(-1, 1, 544).astype(np.float32)
    S.scap_fold_bias_q4(Wq, sc, zero, 128, f32(m), f32(bias), bfg, ws.payload)
    torch.cuda.synchronize()
    bf64 = oracle.fold_bias_q4(d["Wq"], d["scale"], d["zero"], 128, m, bias)
    assert rel_l2_rows(bfg.cpu().numpy(), bf64) <= 1e-6
    y64 = oracle.sparse_fc_q4(xf, d["Wq"], d["scale"], d["zero"], 128, m, 0.3, bf64.astype(np.float32))
    y, _ = run_q4(S, d, m, 0.3, bf64.astype(np.float32), want_idx=False)
    assert rel_l2_rows(y, y64) <= REL_L2_TOL
    yd = torch.empty((5, 544), dtype=torch.float32, device="cuda")
    S.scap_dense_fc_q4(dev(d["x"], si.BF16), Wq, sc, zero, 128, f32(bias), yd, ws.payload)
    torch.cuda.synchronize()
    assert rel_l2_rows(yd.cpu().numpy(), oracle.sparse_fc_q4(xf, d["Wq"], d["scale"], d["zero"], 128, None, 0.0, bias)) <= REL_L2_TOL
    assert ws.intact()


def test_q4_nothing_kept_returns_the_bias_and_rejects_bad_arguments(S):
    d = case(640, 272, 2, si.BF16, 128)
    bf = np.linspace(-1, 1, 272).astype(np.float32)
    y, gidx = run_q4(S, d, d["m_true"], np.inf, bf)
    assert gidx.size == 0 and np.array_equal(y, np.tile(bf, (2, 1)))
    x = dev(d["x"], si.BF16)
    ws = workspace(S.scap_fc_workspace(2, 640, 272))
    yb = torch.empty((2, 272), dtype=torch.float32, device="cuda")
    Wq, zero, sc = torch.from_numpy(d["Wq"]).cuda(), torch.from_numpy(d["zero"]).cuda(), f32(d["scale"])
    with pytest.raises(S.ScapError):  # group not a multiple of 32
        S.scap_sparse_fc_q4(x, Wq, sc, zero, 48, None, f32([0.1]), None, yb, ws.payload)
