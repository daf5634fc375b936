"""scap_calibrate against the oracle: the mode vector and tau must match bit for bit (both sides follow the
same binary32 recipe, and tau is an order statistic interpolated in binary64)."""
import numpy as np
import pytest
import torch

import oracle
import scap_inputs as si
from scap_testlib import dev, workspace

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    import paper_2412_07174_b200 as scap
    scap.lib()
    return scap


def run_calibrate(S, xbits, dt, s, nbins):
    x = dev(xbits, dt)
    T, K = x.shape
    ws = workspace(S.scap_calibrate_workspace(T, K, nbins))
    mg = workspace(K * 4)
    tg = workspace(4)
    m = mg.view(torch.float32, (K,))
    tau = tg.view(torch.float32, (1,))
    S.scap_calibrate(x, s, nbins, m, tau, ws.payload)
    torch.cuda.synchronize()
    assert ws.intact() and mg.intact() and tg.intact()
    return m.cpu().numpy().copy(), np.float32(tau.item())


@pytest.mark.parametrize("T,K,dt,nbins,s", [
    (256, 1024, si.F16, 2048, 0.5),       # config 0's calibration set
    (64, 40, si.BF16, 16, 0.3),           # one partial strip
    (100, 264, si.BF16, 2048, 0.65),
    (513, 72, si.F16, 7, 0.999),
    (32, 8, si.BF16, 1, 0.01),
    (300, 520, si.BF16, 333, 0.8),
])
def test_mode_and_tau_bit_exact(S, T, K, dt, nbins, s):
    d = si.laplace_fc(0 if dt == si.F16 else 4, K, 8, dt, T, 1)
    xf = si.to_f32(d["x_calib"], dt)
    m_o, tau_o = oracle.calibrate(xf, s, nbins)
    m_g, tau_g = run_calibrate(S, d["x_calib"], dt, s, nbins)
    assert np.array_equal(m_g, m_o)
    assert tau_g.view(np.uint32) == np.float32(tau_o).view(np.uint32)


@pytest.mark.parametrize("strip", [16, 32])
@pytest.mark.parametrize("T,K,nbins,s", [
    (2100, 72, 2048, 0.6),    # more rows than a strip keeps in registers: the passes re-read the input
    (300, 520, 333, 0.8),
    (64, 40, 16, 0.3),        # a partial strip for either width
])
def test_both_strip_widths_of_the_histogram_kernel(S, strip, T, K, nbins, s):
    d = si.laplace_fc(4, K, 8, si.BF16, T, 1)
    xf = si.to_f32(d["x_calib"], si.BF16)
    m_o, tau_o = oracle.calibrate(xf, s, nbins)
    S.scap_tune("cal_strip", strip)
    try:
        m_g, tau_g = run_calibrate(S, d["x_calib"], si.BF16, s, nbins)
    finally:
        S.scap_tune("cal_strip", 16)
    assert np.array_equal(m_g, m_o)
    assert tau_g.view(np.uint32) == np.float32(tau_o).view(np.uint32)


def test_no_centring_and_zero_sparsity(S):
    d = si.laplace_fc(4, 128, 8, si.BF16, 200, 1)
    xf = si.to_f32(d["x_calib"], si.BF16)
    m_g, tau_g = run_calibrate(S, d["x_calib"], si.BF16, 0.7, 0)
    assert not m_g.any() and tau_g == oracle.tau(xf, None, 0.7)
    m_g, tau_g = run_calibrate(S, d["x_calib"], si.BF16, 0.0, 64)
    assert np.array_equal(m_g, oracle.mode(xf, 64)) and tau_g == 0.0


def test_constant_channels_and_heavy_ties(S):
    # quantised data: many equal importances, constant channels, both order statistics in one bucket
    T, K = 96, 48
    rng = np.random.default_rng(11)
    x = rng.integers(-3, 4, size=(T, K)).astype(np.float64) * 0.25
    x[:, 5] = 1.5
    x[:, 17] = 0.0
    bits = si.to_bits(x, si.BF16)
    xf = si.to_f32(bits, si.BF16)
    for s in (0.1, 0.5, 0.9):
        for nbins in (4, 2048):
            m_o, tau_o = oracle.calibrate(xf, s, nbins)
            m_g, tau_g = run_calibrate(S, bits, si.BF16, s, nbins)
            assert np.array_equal(m_g, m_o) and tau_g == tau_o


def test_config4_calibration_size(S):
    # 2048 tokens x 14336 channels, 2048 bins: the calibration the sweep times
    d = si.laplace_fc(4, 14336, 8, si.BF16, 2048, 1)
    xf = si.to_f32(d["x_calib"], si.BF16)
    m_o, tau_o = oracle.calibrate(xf, 0.6, 2048)
    m_g, tau_g = run_calibrate(S, d["x_calib"], si.BF16, 0.6, 2048)
    assert np.array_equal(m_g, m_o) and tau_g == tau_o
    keep = oracle.mask(xf[:64], m_o, tau_o)[0]
    assert abs((1 - keep.mean()) - 0.6) < 0.01


# ---------------------------------------------------------------- mean / median estimators and the scalar eta

def run_calibrate_ex(S, xbits, dt, s, estimator, scope, nbins):
    x = dev(xbits, dt)
    T, K = x.shape
    ws = workspace(S.scap_calibrate_workspace(T, K, nbins))
    mg = workspace(K * 4)
    tg = workspace(4)
    m = mg.view(torch.float32, (K,))
    tau = tg.view(torch.float32, (1,))
    S.scap_calibrate_ex(x, s, estimator, scope, nbins, m, tau, ws.payload)
    torch.cuda.synchronize()
    assert ws.intact() and mg.intact() and tg.intact()
    return m.cpu().numpy().copy(), np.float32(tau.item())


@pytest.mark.parametrize("scope", [oracle.PER_CHANNEL, oracle.SCALAR])
@pytest.mark.parametrize("estimator", [oracle.HISTOGRAM, oracle.MEAN, oracle.MEDIAN])
@pytest.mark.parametrize("T,K,dt,nbins,s", [
    (256, 1024, si.F16, 2048, 0.5),
    (64, 40, si.BF16, 16, 0.3),           # one partial strip
    (101, 264, si.BF16, 333, 0.65),       # odd row count: the median is the middle element
    (2500, 72, si.F16, 64, 0.8),          # more rows than a strip keeps in registers
    (1, 8, si.BF16, 4, 0.2),
])
def test_estimators_and_scopes_bit_exact(S, estimator, scope, T, K, dt, nbins, s):
    d = si.laplace_fc(0 if dt == si.F16 else 4, K, 8, dt, T, 1)
    xf = si.to_f32(d["x_calib"], dt)
    m_o, tau_o = oracle.calibrate_ex(xf, s, estimator, scope, nbins)
    m_g, tau_g = run_calibrate_ex(S, d["x_calib"], dt, s, estimator, scope, nbins)
    assert np.array_equal(m_g.view(np.uint32), m_o.view(np.uint32))
    assert tau_g.view(np.uint32) == np.float32(tau_o).view(np.uint32)


@pytest.mark.parametrize("T,K,dt,G,s", [
    (256, 64, si.F16, 129, 0.5),
    (300, 40, si.BF16, 64, 0.3),
    (1000, 16, si.BF16, 2048, 0.7),
    (3, 8, si.BF16, 2, 0.2),
])
def test_kde_peak_matches_the_oracle(S, T, K, dt, G, s):
    # Both sides evaluate the densities in binary64 but with different exp routines and summation orders, so where
    # two grid points are equally dense to within rounding either is right: the mode must be the oracle's, or a grid
    # point whose oracle density is within 1e-9 (relative) of the oracle's maximum.  tau then follows bit for bit.
    d = si.laplace_fc(0 if dt == si.F16 else 4, K, 8, dt, T, 1)
    bits = d["x_calib"].copy()
    bits[:, 3] = bits[0, 3]                               # a constant channel
    xf = si.to_f32(bits, dt)
    m_o = oracle.mode_estimate(xf, oracle.KDE, oracle.PER_CHANNEL, G)
    m_g, tau_g = run_calibrate_ex(S, bits, dt, s, oracle.KDE, oracle.PER_CHANNEL, G)
    differ = np.flatnonzero(m_g.view(np.uint32) != m_o.view(np.uint32))
    assert len(differ) <= max(1, K // 8)
    for k in differ:
        dens, grid = oracle.kde_density(xf, int(k), G)
        i = int(np.flatnonzero(grid.astype(np.float32) == m_g[k])[0])
        assert dens[i] >= dens.max() * (1 - 1e-9)
    assert m_g[3] == xf[0, 3]
    assert tau_g.view(np.uint32) == np.float32(oracle.tau(xf, m_g, s)).view(np.uint32)


def test_kde_rejects_scalar_scope_long_inputs_and_one_point_grids(S):
    L = S.lib()
    P = 0x10000  # never dereferenced: the argument checks come first
    assert L.scap_calibrate_ex(P, 64, 8, 1, 0.5, 3, 1, 64, P, P, P, 1 << 30, None) == 1     # scalar scope: SCAP_ERR_INVALID_ARG
    assert L.scap_calibrate_ex(P, 64, 8, 1, 0.5, 3, 0, 1, P, P, P, 1 << 30, None) == 1      # one grid point
    assert L.scap_calibrate_ex(P, 5000, 8, 1, 0.5, 3, 0, 64, P, P, P, 1 << 30, None) == 2   # T > 4096: SCAP_ERR_SHAPE


def test_skewed_inputs_median_and_mean_differ_from_the_histogram_mode(S):
    # GELU-output-like skew: the three estimators disagree, each matches its oracle, and the better mode prunes more
    rng_bits = si.to_bits(np.abs(si.normal(si.stream_seed(4, 9), 512 * 64).reshape(512, 64)) ** 1.5, si.BF16)
    xf = si.to_f32(rng_bits, si.BF16)
    kept = []
    for est in (oracle.HISTOGRAM, oracle.MEDIAN, oracle.MEAN):
        m_g, _ = run_calibrate_ex(S, rng_bits, si.BF16, 0.5, est, oracle.PER_CHANNEL, 64)
        assert np.array_equal(m_g, oracle.mode_estimate(xf, est, oracle.PER_CHANNEL, 64))
        kept.append(float(np.mean(np.abs(xf - m_g[None, :]) >= np.float32(0.2))))
    assert kept[0] < kept[1] < kept[2]


def test_calibrate_ex_rejects_unknown_estimator_and_scope(S):
    x = dev(si.laplace_fc(4, 64, 8, si.BF16, 16, 1)["x_calib"], si.BF16)
    ws = workspace(S.scap_calibrate_workspace(16, 64, 8))
    m = torch.zeros(64, device="cuda")
    tau = torch.zeros(1, device="cuda")
    for est, scope in ((4, 0), (-1, 0), (0, 2)):
        with pytest.raises(S.ScapError):
            S.scap_calibrate_ex(x, 0.5, est, scope, 8, m, tau, ws.payload)
