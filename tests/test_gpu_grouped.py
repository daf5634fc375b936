"""scap_sparse_fc_grouped: one union mask per caller-named group of rows (Appendix C, overlapping sparsity).  Pruning is
per element, so whatever the grouping every row must equal the oracle's result for that row."""
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


def run_grouped(S, d, m, tau, bf, groups):
    dt = d["dt"]
    x, W = dev(d["x"], dt), dev(d["W"], dt)
    B, K = x.shape
    N = W.shape[1]
    ws = workspace(S.scap_grouped_workspace())
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    y.fill_(float("nan"))
    S.scap_sparse_fc_grouped(x, W, f32(m), f32([tau]), f32(bf), y, groups, ws.payload)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    return y.cpu().numpy().copy()


@pytest.mark.parametrize("K,N,B,n_ctx,groups", [
    (2048, 520, 8, 2, None),                        # two groups of four (FMA bodies inside the tensor-core launch)
    (2048, 520, 16, 2, None),                       # two groups of eight (tensor-core body)
    (1500, 264, 13, 4, None),                       # ragged: groups of 4, 3, 3, 3
    (1024, 1032, 6, 1, [0, 0, 1, 2, 2, 2]),         # caller's own grouping: sizes 2, 1, 3
    (1024, 256, 4, 1, [3, 3, 9, 9]),                # sparse group numbers: groups 0-2, 4-8 are empty
    (4096, 1024, 64, 16, None),                     # 64 rows, 16 groups of four
    (2560, 512, 32, 2, None),                       # two groups of sixteen
])
def test_every_row_matches_the_oracle_whatever_the_grouping(S, K, N, B, n_ctx, groups):
    d = si.context_batch(4, K, N, si.BF16, 64, B, n_ctx, 0.9)
    dt = d["dt"]
    xf = si.to_f32(d["x"], dt)
    m = d["m_true"]
    tau = oracle.tau(si.to_f32(d["x_calib"], dt), m, 0.6)
    bf64 = oracle.fold_bias(d["W"], dt, m, None)
    y64 = oracle.sparse_fc(xf, d["W"], dt, m, tau, None, threads=8) + bf64[None, :]
    y = run_grouped(S, d, m, tau, bf64.astype(np.float32), d["ctx"].tolist() if groups is None else groups)
    assert rel_l2_rows(y, y64) <= REL_L2_TOL


def test_grouped_call_rejects_bad_groupings(S):
    d = si.context_batch(4, 512, 64, si.BF16, 16, 20, 1, 0.5)
    x, W = dev(d["x"], si.BF16), dev(d["W"], si.BF16)
    ws = workspace(S.scap_grouped_workspace())
    y = torch.empty((20, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(S.ScapError):   # 20 rows in one group
        S.scap_sparse_fc_grouped(x, W, None, f32([0.1]), None, y, [0] * 20, ws.payload)
    with pytest.raises(S.ScapError):   # group number out of range
        S.scap_sparse_fc_grouped(x, W, None, f32([0.1]), None, y, [16] + [0] * 19, ws.payload)
