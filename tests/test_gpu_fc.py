"""GPU parity of the sparse FC, the dense baseline and bias folding against the CPU oracle, through the
C ABI.  Mask (kept-channel list) bit-exact; y within 2e-3 relative L2 per row of the oracle's binary64 y."""
import numpy as np
import pytest
import torch

import oracle
import scap_inputs as si
from scap_testlib import REL_L2_TOL, dev, f32, oracle_fc, rel_l2_rows, workspace

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    import paper_2412_07174_b200 as scap
    scap.lib()
    return scap


def run_sparse(S, d, m, tau, bf, x_bits=None, want_idx=True):
    dt = d["dt"]
    x = dev(d["x"] if x_bits is None else x_bits, dt)
    W = dev(d["W"], dt)
    B, K = x.shape
    N = W.shape[1]
    ws = workspace(S.scap_fc_workspace(B, K, N))
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    idx = torch.full((K,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    nnz = torch.full((1,), -1, dtype=torch.int32, device="cuda") if want_idx else None
    S.scap_sparse_fc(x, W, None if m is None else f32(m), f32([tau]), None if bf is None else f32(bf), y, ws.payload,
                     idx_out=idx, nnz_out=nnz)
    torch.cuda.synchronize()
    assert ws.intact() and yg.intact()
    if want_idx:
        n = int(nnz.item())
        return y.cpu().numpy().copy(), idx[:n].cpu().numpy().astype(np.uint32), n
    return y.cpu().numpy().copy(), None, None


def check_fc(S, d, m, tau, with_bias=True):
    dt = d["dt"]
    bf64 = oracle.fold_bias(d["W"], dt, m if m is not None else np.zeros(d["K"], np.float32), d.get("b")) if with_bias else None
    bf32 = None if bf64 is None else bf64.astype(np.float32)
    y64, keep, idx = oracle_fc(d, m, tau, bf64)
    y, gidx, n = run_sparse(S, d, m, tau, bf32)
    assert n == idx.size
    assert np.array_equal(gidx, idx)
    if np.linalg.norm(y64) > 0:
        assert rel_l2_rows(y, y64) <= REL_L2_TOL
    return y, y64, keep


# ---------------------------------------------------------------- config 0 (fp16, 1024 x 1024, batch 1)

def test_config0_single_fc_fp16(S):
    d = si.config0()
    xc = si.to_f32(d["x_calib"], d["dt"])
    m, tau = oracle.calibrate(xc, 0.5, 2048)
    y, y64, keep = check_fc(S, d, m, tau)
    assert 0.3 < keep.mean() < 0.7


# ---------------------------------------------------------------- shapes spanning tiles, ragged tails, batches

@pytest.mark.parametrize("K,N,B,dt", [
    (1000, 264, 1, si.BF16), (33, 8, 3, si.F16), (1, 16, 2, si.BF16), (777, 520, 5, si.BF16),
    (2048, 1032, 16, si.F16), (300, 4096, 4, si.BF16), (5000, 256, 8, si.BF16), (256, 248, 2, si.F16),
    (2560, 10576, 1, si.BF16), (5120, 2560, 4, si.BF16),     # Mamba2-2.7B in_proj / out_proj (N = 10576 ends in a ragged tile)
])
def test_shapes_and_batches(S, K, N, B, dt):
    d = si.laplace_fc(4, K, N, dt, 32, B)
    m = d["m_true"]
    tau = oracle.tau(si.to_f32(d["x_calib"], dt), m, 0.6)
    check_fc(S, d, m, tau)
    check_fc(S, d, None, tau, with_bias=False)


@pytest.mark.parametrize("s", [0.0, 0.25, 0.5, 0.9, 0.99])
def test_sparsity_levels(S, s):
    d = si.laplace_fc(4, 1536, 776, si.BF16, 64, 2)
    m = oracle.mode(si.to_f32(d["x_calib"], d["dt"]), 256)
    tau = oracle.tau(si.to_f32(d["x_calib"], d["dt"]), m, s)
    check_fc(S, d, m, tau)


# ---------------------------------------------------------------- degenerate cases

# the four forms of the kernel a batch of three can run on: (fma_rows, tcgen05, dense_stream) tune values
ROUTES = {"fma": (4, 0, 0), "mma_sync": (2, 0, 0), "tcgen05": (2, 2, 0), "dense_stream": (2, 0, 2)}


def set_route(S, route):
    rows, tc, ds = ROUTES[route]
    S.scap_tune("fma_rows", rows)
    S.scap_tune("tcgen05", tc)
    S.scap_tune("dense_stream", ds)


def reset_route(S):
    S.scap_tune("fma_rows", 4)
    S.scap_tune("tcgen05", 1)
    S.scap_tune("dense_stream", 1)


@pytest.mark.parametrize("route", sorted(ROUTES))
def test_tau_zero_is_dense_and_tau_inf_returns_bias(S, route):
    d = si.laplace_fc(4, 640, 264, si.BF16, 8, 3)
    dt = d["dt"]
    bf = np.linspace(-1, 1, 264).astype(np.float32)
    try:
        set_route(S, route)
        y, idx, n = run_sparse(S, d, None, 0.0, bf)
        assert n == 640 and np.array_equal(idx, np.arange(640, dtype=np.uint32))
        y64 = oracle.dense_fc(si.to_f32(d["x"], dt), d["W"], dt, bf)
        assert rel_l2_rows(y, y64) <= REL_L2_TOL
        y, idx, n = run_sparse(S, d, d["m_true"], np.inf, bf)
        assert n == 0 and np.array_equal(y, np.tile(bf, (3, 1)))   # nnz = 0: y == b_fused exactly
        y, idx, n = run_sparse(S, d, d["m_true"], np.inf, None)
        assert n == 0 and not y.any()
        S.scap_device_status()
    finally:
        reset_route(S)


@pytest.mark.parametrize("route", sorted(ROUTES))
def test_nan_and_threshold_ties_in_a_batch_of_three(S, route):
    K, N = 72, 24
    d = si.laplace_fc(4, K, N, si.BF16, 8, 3)
    x = np.zeros((3, K))
    x[0, 0], x[0, 1], x[0, 2], x[0, 4] = 0.5, -0.5, 0.49, -0.0
    x[1, 5], x[1, 6] = 2.0, -0.25
    x[2, 40], x[2, 71] = -3.0, 0.5
    xb = si.to_bits(x, si.BF16)
    xb[:, 3] = 0x7FC0                                              # bf16 NaN in every row: dropped, never multiplied
    y64, keep, idx = oracle_fc(d, None, 0.5, None, x_bits=xb)
    assert idx.tolist() == [0, 1, 5, 40, 71]
    try:
        set_route(S, route)
        y, gidx, n = run_sparse(S, d, None, 0.5, None, x_bits=xb)
    finally:
        reset_route(S)
    assert gidx.tolist() == [0, 1, 5, 40, 71] and np.isfinite(y).all()
    assert rel_l2_rows(y, y64) <= REL_L2_TOL


def test_ties_signed_zero_and_nan(S):
    K, N = 40, 16
    d = si.laplace_fc(4, K, N, si.BF16, 8, 2)
    x = np.zeros((2, K))
    x[0, 0], x[0, 1], x[0, 2], x[0, 3], x[0, 4] = 0.5, -0.5, 0.49, np.nan, -0.0
    x[1, 5], x[1, 6] = 2.0, -0.25
    xb = si.to_bits(x, si.BF16)
    xb[:, 3] = 0x7FC0                                              # bf16 NaN in both rows
    y64, keep, idx = oracle_fc(d, None, 0.5, None, x_bits=xb)
    assert idx.tolist() == [0, 1, 5]                               # |x| == tau kept; NaN dropped
    y, gidx, n = run_sparse(S, d, None, 0.5, None, x_bits=xb)
    assert gidx.tolist() == [0, 1, 5] and np.isfinite(y).all()
    assert rel_l2_rows(y, y64) <= REL_L2_TOL
    # tau = 0 keeps +-0 too (all channels except the NaN)
    y, gidx, n = run_sparse(S, d, None, 0.0, None, x_bits=xb)
    assert n == K - 1 and 3 not in gidx.tolist() and np.isfinite(y).all()


def test_mask_boundary_uses_one_binary32_subtraction(S):
    # values straddling the threshold by one ulp after the subtraction
    K, N = 512, 64
    d = si.laplace_fc(4, K, N, si.F16, 8, 1)
    m = d["m_true"]
    xf = si.to_f32(d["x"], si.F16)
    dd = np.abs((xf[0] - m).astype(np.float32))
    for t in np.sort(dd)[[10, 100, 300]]:
        for tau in (t, np.nextafter(t, np.float32(np.inf)), np.nextafter(t, np.float32(0))):
            _, keep, idx = oracle_fc(d, m, tau, None)
            _, gidx, n = run_sparse(S, d, m, float(tau), None)
            assert np.array_equal(gidx, idx)


# ---------------------------------------------------------------- properties

def test_bitwise_determinism_and_row_independence(S):
    d = si.laplace_fc(4, 2048, 1024, si.BF16, 16, 4)
    m, tau = d["m_true"], 0.25
    y1, i1, _ = run_sparse(S, d, m, tau, None)
    y2, i2, _ = run_sparse(S, d, m, tau, None)
    assert np.array_equal(y1, y2) and np.array_equal(i1, i2)
    for b in range(4):
        yb, _, _ = run_sparse(S, d, m, tau, None, x_bits=d["x"][b:b + 1])
        y64 = oracle.sparse_fc(si.to_f32(d["x"][b:b + 1], d["dt"]), d["W"], d["dt"], m, tau, None)
        assert rel_l2_rows(yb, y64) <= REL_L2_TOL
        assert rel_l2_rows(y1[b:b + 1], y64) <= REL_L2_TOL


@pytest.mark.parametrize("B", [1, 3, 6, 12])                       # FMA body with 1 and 4 rows, mma.sync with 8 and 16
@pytest.mark.parametrize("split", [1, 2, 3, 4, 5, 6, 7, 8])
def test_any_split_k_gives_the_same_answer(S, split, B):
    # cluster sizes that do not divide the column tile leave the last rank with fewer columns
    d = si.laplace_fc(4, 1500, 520, si.BF16, 16, B)
    try:
        S.scap_tune("split_k", split)
        check_fc(S, d, d["m_true"], 0.2)
    finally:
        S.scap_tune("split_k", 0)


def test_pdl_off_gives_identical_bits(S):
    d = si.laplace_fc(4, 1500, 520, si.BF16, 16, 2)
    y1, _, _ = run_sparse(S, d, d["m_true"], 0.2, None)
    try:
        S.scap_tune("pdl", 0)
        y2, _, _ = run_sparse(S, d, d["m_true"], 0.2, None)
    finally:
        S.scap_tune("pdl", 1)
    assert np.array_equal(y1, y2)


@pytest.mark.parametrize("B", [1, 2, 4])
@pytest.mark.parametrize("chunks", [1, 6, 64])
def test_early_row_hints_change_no_bit(S, B, chunks):
    """The optional L2 hints for the head of a sparse call's row stream (tune key head_rows) are requests without a
    result: the kept list and every output bit stay as they are, also when the hint reaches past the rank's channels."""
    d = si.laplace_fc(B, 1500, 520, si.BF16, 16, 2)
    y1, idx1, nnz1 = run_sparse(S, d, d["m_true"], 0.2, None)
    try:
        S.scap_tune("head_rows", chunks)
        y2, idx2, nnz2 = run_sparse(S, d, d["m_true"], 0.2, None)
    finally:
        S.scap_tune("head_rows", 0)
    assert nnz1 == nnz2 and np.array_equal(idx1, idx2)
    assert np.array_equal(y1, y2)
    with pytest.raises(Exception):
        S.scap_tune("head_rows", 65)


def test_back_to_back_calls_share_a_workspace(S):
    # many calls in a row on one stream with different inputs: each must see only its own lists
    d = si.laplace_fc(4, 1024, 512, si.BF16, 16, 8)
    dt = d["dt"]
    W = dev(d["W"], dt)
    m = f32(d["m_true"])
    tau = f32([0.3])
    ws = workspace(S.scap_fc_workspace(1, 1024, 512))
    xs = [dev(d["x"][b:b + 1], dt) for b in range(8)]
    ys = [torch.empty((1, 512), dtype=torch.float32, device="cuda") for _ in range(8)]
    for rep in range(3):
        for b in range(8):
            S.scap_sparse_fc(xs[b], W, m, tau, None, ys[b], ws.payload)
    torch.cuda.synchronize()
    assert ws.intact()
    for b in range(8):
        y64 = oracle.sparse_fc(si.to_f32(d["x"][b:b + 1], dt), d["W"], dt, d["m_true"], 0.3, None)
        assert rel_l2_rows(ys[b].cpu().numpy(), y64) <= REL_L2_TOL


def test_cuda_graph_replay_matches_eager(S):
    d = si.laplace_fc(4, 1024, 512, si.BF16, 16, 2)
    dt = d["dt"]
    x, W, m, tau = dev(d["x"], dt), dev(d["W"], dt), f32(d["m_true"]), f32([0.3])
    ws = workspace(S.scap_fc_workspace(2, 1024, 512))
    y_e = torch.empty((2, 512), dtype=torch.float32, device="cuda")
    y_g = torch.zeros((2, 512), dtype=torch.float32, device="cuda")
    S.scap_sparse_fc(x, W, m, tau, None, y_e, ws.payload)
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            S.scap_sparse_fc(x, W, m, tau, None, y_g, ws.payload)
            S.scap_sparse_fc(x, W, m, tau, None, y_g, ws.payload)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(y_e, y_g)


# ---------------------------------------------------------------- dense baseline, bias folding, host variant

@pytest.mark.parametrize("K,N,B,dt", [(1000, 264, 1, si.BF16), (2048, 1032, 16, si.F16), (640, 4096, 3, si.BF16)])
def test_dense_fc(S, K, N, B, dt):
    d = si.laplace_fc(4, K, N, dt, 8, B)
    x, W = dev(d["x"], dt), dev(d["W"], dt)
    b = np.linspace(-2, 2, N).astype(np.float32)
    ws = workspace(S.scap_fc_workspace(B, K, N))
    yg = workspace(B * N * 4)
    y = yg.view(torch.float32, (B, N))
    S.scap_dense_fc(x, W, f32(b), y, ws.payload)
    assert ws.intact() and yg.intact()
    y64 = oracle.dense_fc(si.to_f32(d["x"], dt), d["W"], dt, b)
    assert rel_l2_rows(y.cpu().numpy(), y64) <= REL_L2_TOL
    S.scap_dense_fc(x, W, None, y, ws.payload)
    torch.cuda.synchronize()
    assert rel_l2_rows(y.cpu().numpy(), oracle.dense_fc(si.to_f32(d["x"], dt), d["W"], dt, None)) <= REL_L2_TOL


@pytest.mark.parametrize("K,N,dt,bias", [(1024, 1024, si.F16, True), (1000, 264, si.BF16, False), (4096, 520, si.BF16, True)])
def test_fold_bias(S, K, N, dt, bias):
    d = si.laplace_fc(0, K, N, dt, 8, 1, with_bias=bias)
    W = dev(d["W"], dt)
    m = d["m_true"]
    b = dev(d["b"], dt) if bias else None
    ws = workspace(S.scap_fold_bias_workspace(K, N))
    og = workspace(N * 4)
    out = og.view(torch.float32, (N,))
    S.scap_fold_bias(W, f32(m), b, out, ws.payload)
    assert ws.intact() and og.intact()
    want = oracle.fold_bias(d["W"], dt, m, d["b"])
    got = out.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-6


@pytest.mark.parametrize("pinned,direct", [(True, 1), (True, 0), (False, 1)])
@pytest.mark.parametrize("B", [1, 4])
def test_host_buffer_variant_matches_device_variant(S, pinned, direct, B):
    # pinned + direct: the library's kernels pull x from and store y to host memory; otherwise staging copies
    d = si.laplace_fc(4, 1024, 520, si.BF16, 16, B)
    dt = d["dt"]
    y_dev, _, _ = run_sparse(S, d, d["m_true"], 0.3, None, want_idx=False)
    W, m, tau = dev(d["W"], dt), f32(d["m_true"]), f32([0.3])
    xh = si.as_torch(d["x"], dt)
    yh = torch.zeros((B, 520), dtype=torch.float32)
    if pinned:
        xh, yh = xh.pin_memory(), yh.pin_memory()
    ws = workspace(S.scap_fc_host_workspace(B, 1024, 520))
    try:
        S.scap_tune("host_direct", direct)
        S.scap_sparse_fc_host(xh, W, m, tau, None, yh, ws.payload)
        torch.cuda.synchronize()
    finally:
        S.scap_tune("host_direct", 1)
    assert ws.intact()
    assert np.array_equal(yh.numpy(), y_dev)


# ---------------------------------------------------------------- batch 3..16 on the tcgen05 kernel (forced)

@pytest.mark.parametrize("K,N,B,dt,split", [
    (1500, 520, 3, si.BF16, 0), (1500, 520, 4, si.BF16, 3), (2048, 1024, 8, si.BF16, 0), (4100, 264, 5, si.F16, 0),
    (1024, 136, 12, si.F16, 2), (3000, 640, 16, si.BF16, 0), (96, 8, 7, si.BF16, 1), (6000, 256, 9, si.BF16, 1),
])
def test_tcgen05_kernel_matches_the_oracle(S, K, N, B, dt, split):
    # several fills of the operand region (6000 channels in one CTA), ragged tiles, both dtypes, all row groupings
    d = si.laplace_fc(4, K, N, dt, 16, B)
    try:
        S.scap_tune("tcgen05", 2)
        S.scap_tune("dense_stream", 0)
        S.scap_tune("split_k", split)
        check_fc(S, d, d["m_true"], 0.25)
        check_fc(S, d, None, 0.4, with_bias=False)
        S.scap_device_status()
    finally:
        S.scap_tune("tcgen05", 1)
        S.scap_tune("dense_stream", 1)
        S.scap_tune("split_k", 0)


@pytest.mark.parametrize("K,N,B,dt", [(777, 520, 3, si.BF16), (300, 4096, 4, si.BF16), (2048, 1032, 4, si.F16), (33, 8, 3, si.F16)])
def test_batch_three_and_four_on_the_mma_sync_route(S, K, N, B, dt):
    d = si.laplace_fc(4, K, N, dt, 32, B)
    tau = oracle.tau(si.to_f32(d["x_calib"], dt), d["m_true"], 0.6)
    try:
        set_route(S, "mma_sync")
        check_fc(S, d, d["m_true"], tau)
    finally:
        reset_route(S)


def test_tcgen05_and_mma_sync_paths_agree_closely(S):
    d = si.laplace_fc(4, 2048, 512, si.BF16, 16, 6)
    ys = []
    for mode in (0, 2):
        try:
            S.scap_tune("tcgen05", mode)
            ys.append(run_sparse(S, d, d["m_true"], 0.3, None)[0])
        finally:
            S.scap_tune("tcgen05", 1)
    assert rel_l2_rows(ys[1], ys[0].astype(np.float64)) <= 1e-6


# ---------------------------------------------------------------- parameters produced on the stream right before the call

@pytest.mark.parametrize("B", [1, 4, 8])
def test_parameters_rewritten_on_the_stream_directly_before_the_call(S, B):
    """tau, m and the fused bias are rewritten by ordinary kernels (device copies and a fill) and the sparse FC is enqueued at
    once on the same stream, several times over with alternating parameter sets and no synchronisation in between:
    every call must see the values written just before it (kept list bit-exact, y within tolerance)."""
    K, N = 2048, 1032
    d = si.laplace_fc(4, K, N, si.BF16, 32, B)
    dt = d["dt"]
    xf = si.to_f32(d["x"], dt)
    xcf = si.to_f32(d["x_calib"], dt)
    sets = []
    for i, (shift, s) in enumerate([(0.0, 0.5), (0.07, 0.8), (-0.05, 0.3)]):
        m = (d["m_true"] + np.float32(shift)).astype(np.float32)
        tau = oracle.tau(xcf, m, s)
        bf64 = oracle.fold_bias(d["W"], dt, m, d.get("b"))
        sets.append((m, float(tau), bf64))
    x, W = dev(d["x"], dt), dev(d["W"], dt)
    m_src = [f32(m) for m, _, _ in sets]
    b_src = [f32(bf.astype(np.float32)) for _, _, bf in sets]
    m_dev, b_dev = torch.empty_like(m_src[0]), torch.empty_like(b_src[0])
    tau_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = workspace(S.scap_fc_workspace(B, K, N))
    rounds = 9
    ys = [torch.empty((B, N), dtype=torch.float32, device="cuda") for _ in range(rounds)]
    idxs = [torch.full((K,), -1, dtype=torch.int32, device="cuda") for _ in range(rounds)]
    nnzs = [torch.full((1,), -1, dtype=torch.int32, device="cuda") for _ in range(rounds)]
    S.scap_tune("pdl", 1)
    for r in range(rounds):
        i = r % len(sets)
        m_dev.copy_(m_src[i])           # device-to-device copy kernels and a fill kernel on the current stream ...
        b_dev.copy_(b_src[i])
        tau_dev.fill_(sets[i][1])
        S.scap_sparse_fc(x, W, m_dev, tau_dev, b_dev, ys[r], ws.payload, idx_out=idxs[r], nnz_out=nnzs[r])  # ... and the call, at once
    torch.cuda.synchronize()
    assert ws.intact()
    for r in range(rounds):
        m, tau, bf64 = sets[r % len(sets)]
        y64 = oracle.sparse_fc(xf, d["W"], dt, m, tau, None) + bf64[None, :]
        idx_o = oracle.mask(xf, m, tau)[2]
        n = int(nnzs[r].item())
        assert n == idx_o.size and np.array_equal(idxs[r][:n].cpu().numpy().astype(np.uint32), idx_o), "round %d" % r
        assert rel_l2_rows(ys[r].cpu().numpy(), y64) <= REL_L2_TOL


# ---------------------------------------------------------------- the bounded waits of the tcgen05 kernel can run out

@pytest.mark.parametrize("kernel", ["gather", "dense_stream"])
def test_a_wait_that_runs_out_is_reported_once_and_the_next_call_is_correct(S, kernel):
    """With the poll limit of the tcgen05 kernels' barrier waits set to 1 the waits of the next call give up at once:
    the call must still return (every CTA passes its cluster barriers and frees its tensor memory),
    scap_device_status must report the time-out exactly once, and an ordinary call afterwards must pass parity."""
    from paper_2412_07174_b200 import ScapError
    K, N, B = 2048, 512, 5
    d = si.laplace_fc(4, K, N, si.BF16, 32, B)
    m = d["m_true"]
    tau = oracle.tau(si.to_f32(d["x_calib"], d["dt"]), m, 0.5)
    try:
        S.scap_tune("tcgen05", 2)      # batch 5 on the gather tcgen05 kernel, or on the dense-stream one
        S.scap_tune("dense_stream", 2 if kernel == "dense_stream" else 0)
        S.scap_device_status()         # clean slate (raises if an earlier test left a record)
        S.scap_tune("tc_spin", 1)
        run_sparse(S, d, m, tau, None, want_idx=False)   # returns; y is incomplete and not looked at
        with pytest.raises(ScapError) as err:
            S.scap_device_status()
        assert err.value.code == 7     # SCAP_ERR_TIMEOUT
        S.scap_device_status()         # reported once: the record is cleared
        S.scap_tune("tc_spin", 0)
        check_fc(S, d, m, tau)         # the same kernel with its normal limit
        S.scap_device_status()
    finally:
        S.scap_tune("tc_spin", 0)
        S.scap_tune("tcgen05", 1)
        S.scap_tune("dense_stream", 1)


# ---------------------------------------------------------------- batch 3..16 on the dense-stream tcgen05 kernel (forced)

@pytest.mark.parametrize("K,N,B,dt,split", [
    (2048, 512, 8, si.BF16, 0), (2048, 512, 16, si.BF16, 0), (1000, 264, 5, si.BF16, 0), (777, 520, 3, si.F16, 0),
    (4096, 1032, 12, si.F16, 0), (640, 128, 16, si.BF16, 1), (2500, 256, 7, si.BF16, 3), (11008, 4096, 8, si.BF16, 0),
    (64, 16, 4, si.BF16, 0), (100, 2048, 9, si.F16, 0),
])
def test_dense_stream_kernel_matches_the_oracle(S, K, N, B, dt, split):
    """Every row of W is streamed with TMA box loads and pruning happens on the activation operand: same results as the
    gather kernels (kept list bit-exact, y within tolerance), for ragged K (not a multiple of 64), ragged N and all cluster sizes."""
    d = si.laplace_fc(4, K, N, dt, 32, B)
    m = d["m_true"]
    tau = oracle.tau(si.to_f32(d["x_calib"], dt), m, 0.6)
    try:
        S.scap_tune("dense_stream", 2)
        S.scap_tune("split_k", split)
        check_fc(S, d, m, tau)
        check_fc(S, d, None, 0.0, with_bias=False)
        S.scap_device_status()
    finally:
        S.scap_tune("dense_stream", 1)
        S.scap_tune("split_k", 0)
