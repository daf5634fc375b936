"""Pins for the CPU oracle: each check ties one oracle function to something other than itself
(a closed form, a hand-worked case, brute force, a textbook/library special case, or a value the
paper prints), chosen so that a dropped term, a wrong sign or index or a transposed operand fails."""
import math
import os

import numpy as np
import pytest

import oracle
import scap_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rel_l2(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def small_fc(K=96, N=40, B=3, dt=si.BF16, cfg=0):
    return si.laplace_fc(cfg, K, N, dt, 64, B)


# ------------------------------------------------------------------ widening

@pytest.mark.parametrize("dt", [si.F16, si.BF16])
def test_widen_every_pattern_matches_independent_widening(dt):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    a = oracle.widen(bits, dt)
    b = si.to_f32(bits, dt)
    nan = np.isnan(b)
    assert np.array_equal(np.isnan(a), nan)
    assert np.array_equal(a[~nan].view(np.uint32), b[~nan].view(np.uint32))


# ------------------------------------------------------------------ mask (Eq. 2, Alg. 3)

def test_mask_hand_worked_case():
    # x - m by hand: [0.5-0.25, -1-0, 0.125-0.125, 2-3, 0.75-0.5] = [0.25, -1, 0, -1, 0.25]; tau = 0.25
    x = np.array([[0.5, -1.0, 0.125, 2.0, 0.75]], np.float32)
    m = np.array([0.25, 0.0, 0.125, 3.0, 0.5], np.float32)
    keep, U, idx, d = oracle.mask(x, m, 0.25, want_d=True)
    assert keep.tolist() == [[True, True, False, True, True]]      # |d| == tau is kept (Alg. 3: >=)
    assert idx.tolist() == [0, 1, 3, 4]
    assert d.tolist() == [[0.25, -1.0, 0.0, -1.0, 0.25]]
    keep, U, idx = oracle.mask(x, m, np.nextafter(np.float32(0.25), np.float32(1)))
    assert keep.tolist() == [[False, True, False, True, False]]


def test_mask_union_over_batch_and_sorted_idx():
    x = np.array([[1.0, 0.0, 0.0, 0.1], [0.0, 0.0, 2.0, 0.1], [0.0, 0.0, 0.0, 0.1]], np.float32)
    keep, U, idx = oracle.mask(x, None, 0.5)
    assert U.tolist() == [True, False, True, False]
    assert idx.tolist() == [0, 2]
    assert keep.sum() == 2


def test_mask_tau_zero_keeps_all_inf_keeps_none_nan_dropped():
    x = np.array([[0.0, -0.0, 1e-30, np.nan, -5.0]], np.float32)
    keep, _, idx = oracle.mask(x, None, 0.0)
    assert keep.tolist() == [[True, True, True, False, True]]      # +-0 kept at tau = 0; NaN compares false
    keep, _, idx = oracle.mask(x, None, np.inf)
    assert not keep.any() and idx.size == 0


def test_mask_uses_single_binary32_subtraction():
    # 1 + 2^-24 is not a binary32 number; x - m must round to binary32 before the compare.
    x = np.array([[1.0]], np.float32)
    m = np.array([-2.0 ** -25], np.float32)                        # exact difference 1 + 2^-25 rounds to 1.0f
    tau = np.nextafter(np.float32(1.0), np.float32(2.0))           # smallest float above 1
    assert not oracle.mask(x, m, tau)[0].any()                     # rounded d = 1.0 < tau
    assert oracle.mask(x, m, np.float32(1.0))[0].all()


def test_masks_are_nested_as_tau_grows():
    d = small_fc()
    xf = si.to_f32(d["x"], d["dt"])
    prev = None
    for t in [0.0, 0.05, 0.2, 0.5, 1.0, 3.0]:
        keep = oracle.mask(xf, d["m_true"], t)[0]
        if prev is not None:
            assert not (keep & ~prev).any()
        prev = keep


# ------------------------------------------------------------------ sparse FC (Eq. 3)

def brute_force_fc(xf, Wf, m, tau, bf):
    """Pure-Python statement: zero the pruned entries of x - m, then a dense product, fsum-accumulated."""
    B, K = xf.shape
    N = Wf.shape[1]
    y = np.zeros((B, N))
    for b in range(B):
        xp = []
        for k in range(K):
            d32 = np.float32(xf[b, k]) - (np.float32(m[k]) if m is not None else np.float32(0))
            kept = abs(float(d32)) >= float(np.float32(tau))
            xp.append((float(xf[b, k]) - (float(m[k]) if m is not None else 0.0)) if kept else 0.0)
        for n in range(N):
            y[b, n] = math.fsum([xp[k] * float(Wf[k, n]) for k in range(K)] + [float(bf[n]) if bf is not None else 0.0])
    return y


@pytest.mark.parametrize("dt", [si.F16, si.BF16])
def test_sparse_fc_matches_brute_force_on_tiny_shapes(dt):
    d = si.laplace_fc(0, 13, 7, dt, 8, 3)
    xf, Wf = si.to_f32(d["x"], dt), si.to_f32(d["W"], dt)
    bf = np.linspace(-1, 1, 7).astype(np.float32)
    for tau in [0.0, 0.1, 0.3, 10.0]:
        y = oracle.sparse_fc(xf, d["W"], dt, d["m_true"], tau, bf)
        yb = brute_force_fc(xf, Wf, d["m_true"], tau, bf)
        assert np.allclose(y, yb, rtol=1e-13, atol=1e-15)
        y2 = oracle.sparse_fc(xf, d["W"], dt, None, tau, None)
        assert np.allclose(y2, brute_force_fc(xf, Wf, None, tau, None), rtol=1e-13, atol=1e-15)


def test_sparse_fc_tau_zero_is_the_textbook_gemm():
    d = small_fc(K=200, N=72, B=4)
    dt = d["dt"]
    xf, Wf = si.to_f32(d["x"], dt).astype(np.float64), si.to_f32(d["W"], dt).astype(np.float64)
    b = np.arange(72, dtype=np.float32) * 0.01
    y = oracle.sparse_fc(xf, d["W"], dt, None, 0.0, b)
    assert rel_l2(y, xf @ Wf + b) < 1e-14
    assert rel_l2(oracle.dense_fc(xf, d["W"], dt, b), xf @ Wf + b) < 1e-14
    # a transposed weight would change the shape of the product; a wrong row stride would change values
    m = d["m_true"]
    y = oracle.sparse_fc(xf, d["W"], dt, m, 0.0, b)
    assert rel_l2(y, (xf - m.astype(np.float64)) @ Wf + b) < 1e-14


def test_sparse_fc_tau_inf_returns_fused_bias_exactly():
    d = small_fc()
    bf = np.linspace(-3, 3, d["N"]).astype(np.float32)
    y = oracle.sparse_fc(si.to_f32(d["x"], d["dt"]), d["W"], d["dt"], d["m_true"], np.inf, bf)
    assert np.array_equal(y, np.tile(bf.astype(np.float64), (3, 1)))


def test_sparse_fc_rows_are_independent_per_element_pruning():
    d = small_fc(B=5)
    xf = si.to_f32(d["x"], d["dt"])
    yB = oracle.sparse_fc(xf, d["W"], d["dt"], d["m_true"], 0.2, None)
    for b in range(5):
        y1 = oracle.sparse_fc(xf[b:b + 1], d["W"], d["dt"], d["m_true"], 0.2, None)
        assert np.array_equal(yB[b], y1[0])


def test_sparse_fc_column_ranges_threads_and_full_form_agree():
    d = small_fc(K=64, N=50, B=2)
    xf = si.to_f32(d["x"], d["dt"])
    args = (xf, d["W"], d["dt"], d["m_true"], 0.15, np.ones(50, np.float32))
    y = oracle.sparse_fc_full(*args)
    assert np.array_equal(oracle.sparse_fc(*args), y)
    assert np.array_equal(oracle.sparse_fc(*args, threads=3), y)
    assert np.array_equal(oracle.sparse_fc(*args, cols=(7, 31)), y[:, 7:31])


def test_sparse_fc_equals_explicit_mask_times_dense():
    d = small_fc(K=128, N=24, B=2)
    dt = d["dt"]
    xf = si.to_f32(d["x"], dt)
    m = d["m_true"]
    keep, _, _ = oracle.mask(xf, m, 0.25)
    xp = np.where(keep, xf.astype(np.float64) - m.astype(np.float64), 0.0)
    y = oracle.sparse_fc(xf, d["W"], dt, m, 0.25, None)
    assert rel_l2(y, xp @ si.to_f32(d["W"], dt).astype(np.float64)) < 1e-14
    assert 0.2 < keep.mean() < 0.8


# ------------------------------------------------------------------ bias folding (Eq. 4-6)

def test_fold_bias_identity_centred_fc_equals_plain_fc():
    d = small_fc(K=300, N=33, B=2, dt=si.F16)
    dt = d["dt"]
    xf = si.to_f32(d["x"], dt)
    m = d["m_true"]
    bf64 = oracle.fold_bias(d["W"], dt, m, d["b"])
    plain = oracle.dense_fc(xf, d["W"], dt, si.to_f32(d["b"], dt))
    # centred FC at tau = 0 without bias, plus the folded bias kept in float64
    centred = oracle.sparse_fc(xf, d["W"], dt, m, 0.0, None) + bf64[None, :]
    assert rel_l2(centred, plain) < 1e-12


def test_fold_bias_scalar_mode_is_eta_times_column_sum():
    d = small_fc(K=77, N=19)
    dt = d["dt"]
    Wf = si.to_f32(d["W"], dt).astype(np.float64)
    eta = np.float32(0.375)
    bf = oracle.fold_bias(d["W"], dt, np.full(77, eta, np.float32), d["b"])
    assert np.allclose(bf, si.to_f32(d["b"], dt) + float(eta) * Wf.sum(axis=0), rtol=1e-13, atol=1e-15)
    assert np.allclose(oracle.fold_bias(d["W"], dt, np.full(77, eta, np.float32), None), float(eta) * Wf.sum(axis=0),
                       rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------ threshold (Eq. 2 quantile)

@pytest.mark.parametrize("s", [0.05, 0.3, 0.5, 0.731, 0.9, 0.999])
def test_tau_matches_library_linear_quantile(s):
    d = small_fc(K=101, N=8)
    xc = si.to_f32(d["x_calib"], d["dt"])
    m = d["m_true"]
    v = np.abs((xc - m[None, :]).astype(np.float32)).ravel()
    want = np.float32(np.quantile(v.astype(np.float64), s, method="linear"))
    got = oracle.tau(xc, m, s)
    assert abs(float(got) - float(want)) <= float(np.spacing(want))


def test_tau_hand_worked_and_degenerate():
    x = np.array([[4.0, -1.0], [2.0, -3.0]], np.float32)           # |x| sorted: 1 2 3 4
    assert oracle.tau(x, None, 0.5) == np.float32(2.5)             # pos = 1.5
    assert oracle.tau(x, None, 1.0 / 3.0) == np.float32(2.0)       # pos = 1 exactly
    assert oracle.tau(x, None, 0.0) == np.float32(0.0)
    assert oracle.tau(x, None, -1.0) == np.float32(0.0)
    t, vj, vj1 = oracle.tau(x, None, 0.75, want_neighbours=True)   # pos = 2.25
    assert (t, vj, vj1) == (np.float32(3.25), np.float32(3.0), np.float32(4.0))
    m = np.array([1.0, -1.0], np.float32)                          # |x - m| = 3 0 1 2
    assert oracle.tau(x, m, 0.5) == np.float32(1.5)


def test_tau_closed_form_for_laplace_importance():
    # |x - m| ~ Exp(1/b) when x = m + Laplace(0, b): quantile(s) = -b ln(1 - s)  (0.2079 at s = 0.5, b = 0.3)
    d = si.config0()
    xc = si.to_f32(d["x_calib"], d["dt"])
    for s in [0.25, 0.5, 0.8]:
        t = float(oracle.tau(xc, d["m_true"], s))
        assert abs(t / (-0.3 * math.log(1 - s)) - 1) < 0.02


@pytest.mark.parametrize("s", [0.3, 0.5, 0.65, 0.8])
def test_dropped_fraction_on_calibration_set_equals_target(s):
    d = small_fc(K=256, N=8)
    xc = si.to_f32(d["x_calib"], d["dt"])
    m = oracle.mode(xc, 64)
    t = oracle.tau(xc, m, s)
    keep = oracle.mask(xc, m, t)[0]
    M = keep.size
    ties = int((np.abs((xc - m[None, :]).astype(np.float32)) == t).sum())
    assert abs((1.0 - keep.mean()) - s) <= (2 + ties) / M


def test_kept_fraction_on_fresh_data_within_binomial_error():
    # Eq. 2's reading: tau = Quantile(|X_calib|, s) "is expected to yield" sparsity s on new data.
    d = si.laplace_fc(0, 2048, 8, si.BF16, 512, 8)
    xc, xt = si.to_f32(d["x_calib"], d["dt"]), si.to_f32(d["x"], d["dt"])
    s = 0.6
    t = oracle.tau(xc, d["m_true"], s)
    keep = oracle.mask(xt, d["m_true"], t)[0]
    sigma = math.sqrt(s * (1 - s) / keep.size + s * (1 - s) / xc.size)
    assert abs((1 - keep.mean()) - s) < 4 * sigma


# ------------------------------------------------------------------ mode (histogram arg-max)

def test_mode_hand_built_cases():
    # channel 0: 8 samples, 4 bins over [0, 4): bins hold {0, .5}, {1.5}, {2.1, 2.2, 2.9}, {3.9, 4(max -> last)}
    c0 = [0.0, 0.5, 1.5, 2.1, 2.2, 2.9, 3.9, 4.0]
    # channel 1: constant
    c1 = [0.75] * 8
    # channel 2: tie between bin 0 and bin 3 -> lowest bin wins.  range [-1, 1], width 0.5
    c2 = [-1.0, -0.9, -0.8, 0.1, 0.6, 0.7, 1.0, -0.3]
    x = np.array([c0, c1, c2], np.float32).T.copy()
    m = oracle.mode(x, 4)
    assert m[0] == np.float32(2.5)                                  # centre of bin 2 = 0 + 2.5 * 1.0
    assert m[1] == np.float32(0.75)
    assert m[2] == np.float32(-0.75)                                # centre of bin 0 = -1 + 0.5 * 0.5


def test_mode_recovers_planted_per_channel_mode():
    d = si.config0()
    xc = si.to_f32(d["x_calib"], d["dt"])
    m = oracle.mode(xc, 2048)
    err = np.abs(m - d["m_true"])
    assert np.median(err) < 0.1
    # a coarser histogram is a much better estimator at 256 samples; it must land close
    assert np.median(np.abs(oracle.mode(xc, 32) - d["m_true"])) < 0.06


def test_mode_is_translation_equivariant_on_exact_grid():
    # values on a dyadic grid: shifting every sample by 2 shifts the estimate by exactly 2
    rng = np.random.default_rng(5)
    x = (rng.integers(0, 64, size=(200, 6)) / 16.0).astype(np.float32)
    assert np.array_equal(oracle.mode(x + np.float32(2.0), 16), oracle.mode(x, 16) + np.float32(2.0))


def test_mode_matches_the_library_histogram_away_from_bin_edges():
    # Samples at exact bin centres of [0, 64) plus the two range ends: every bin decision is exact in any arithmetic,
    # so numpy.histogram (float64 edges) must count what the oracle counts, and the first arg-max bin centre is the mode.
    rng = np.random.default_rng(17)
    T, K, nbins = 500, 9, 64
    bins = rng.integers(0, nbins, size=(T, K))
    bins[:60, 3] = 41                       # a clear peak
    bins[:40, 4] = 7
    bins[40:80, 4] = 50                     # two tall peaks; whichever is taller (or the lower bin on a tie) must win
    x = (bins + 0.5).astype(np.float32)
    x[-1, :] = 0.0                          # range ends: lo = 0 (bin 0), hi = 64 (clamped into the last bin)
    x[-2, :] = 64.0
    m = oracle.mode(x, nbins)
    for k in range(K):
        counts, edges = np.histogram(x[:, k].astype(np.float64), bins=nbins, range=(0.0, 64.0))
        i = int(np.argmax(counts))          # first maximum = lowest bin
        assert m[k] == np.float32(0.5 * (edges[i] + edges[i + 1]))


def test_calibrate_runs_mode_then_tau_on_centred_values():
    d = small_fc(K=64, N=8)
    xc = si.to_f32(d["x_calib"], d["dt"])
    m, t = oracle.calibrate(xc, 0.5, 16)
    assert np.array_equal(m, oracle.mode(xc, 16)) and t == oracle.tau(xc, m, 0.5)
    m0, t0 = oracle.calibrate(xc, 0.5, 0)
    assert not m0.any() and t0 == oracle.tau(xc, None, 0.5)
    # centring on the planted mode lowers the threshold needed for the same sparsity (Section 3's point)
    assert oracle.tau(xc, d["m_true"], 0.5) < t0


# ------------------------------------------------------------------ SwiGLU block (Alg. 2)

def tiny_glu(D=48, F=80, B=3, cfg=2):
    return si.glu_block(cfg, D, F, si.BF16, 32, B)


def test_glu_all_tau_zero_is_dense_swiglu():
    g = tiny_glu()
    dt = g["dt"]
    hf = si.to_f32(g["h"], dt).astype(np.float64)
    Wgu, Wd = si.to_f32(g["Wgu"], dt).astype(np.float64), si.to_f32(g["Wd"], dt).astype(np.float64)
    F = g["F"]
    gu = hf @ Wgu
    z = gu[:, F:] * (gu[:, :F] / (1 + np.exp(-gu[:, :F])))            # up * silu(gate)
    y, z32 = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, None, 0.0, None, None, 0.0, None)
    assert np.array_equal(z32, z.astype(np.float32))
    assert rel_l2(y, z.astype(np.float32).astype(np.float64) @ Wd) < 1e-13
    # swapping the gate and up halves must change the result (silu is applied to the gate half only)
    z_swapped = gu[:, :F] * (gu[:, F:] / (1 + np.exp(-gu[:, F:])))
    assert rel_l2(z32, z_swapped) > 0.1


def test_glu_stagewise_composition_and_teacher_forcing():
    g = tiny_glu()
    dt = g["dt"]
    hf = si.to_f32(g["h"], dt)
    D, F = g["D"], g["F"]
    m1 = np.linspace(-0.2, 0.2, D).astype(np.float32)
    m2 = np.full(F, 0.001, np.float32)
    b1 = oracle.fold_bias(g["Wgu"], dt, m1, None).astype(np.float32)
    b2 = oracle.fold_bias(g["Wd"], dt, m2, None).astype(np.float32)
    y, z = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, m1, 0.4, b1, m2, 0.01, b2)
    gu = oracle.sparse_fc(hf, g["Wgu"], dt, m1, 0.4, b1)
    z_ref = (gu[:, F:] * (gu[:, :F] / (1 + np.exp(-gu[:, :F])))).astype(np.float32)
    assert np.array_equal(z, z_ref)
    assert np.array_equal(y, oracle.sparse_fc(z, g["Wd"], dt, m2, 0.01, b2))
    # teacher forcing: a supplied z replaces the computed one
    z2 = (z * np.float32(0.5)).astype(np.float32)
    y2, zo = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, m1, 0.4, b1, m2, 0.01, b2, z_in=z2)
    assert np.array_equal(zo, z2)
    assert np.array_equal(y2, oracle.sparse_fc(z2, g["Wd"], dt, m2, 0.01, b2))
    # stage 2 really prunes: some but not all channels kept
    k2 = oracle.mask(z, m2, 0.01)[0]
    assert 0.05 < k2.mean() < 0.95


def test_glu_stage1_batch_agrees_with_loop_form():
    g = tiny_glu(B=6)
    dt = g["dt"]
    hf = si.to_f32(g["h"], dt)
    m1 = np.linspace(-0.1, 0.1, g["D"]).astype(np.float32)
    b1 = oracle.fold_bias(g["Wgu"], dt, m1, None).astype(np.float32)
    _, z = oracle.glu_ffn(hf, g["Wgu"], g["Wd"], dt, m1, 0.3, b1, None, 0.0, None)
    zb = oracle.glu_stage1_batch(hf, g["Wgu"], dt, m1, 0.3, b1)
    assert np.allclose(zb, z, rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------ MoE (router convention: unpinned by the paper)

def test_router_brute_force_ties_and_normalisation():
    lg = np.array([[0.1, 2.0, -1.0, 2.0, 0.5], [3.0, 3.0, 3.0, 3.0, 3.0], [-5.0, 0.0, 1.0, 0.5, 0.9]], np.float32)
    ex, w = oracle.router(lg, 2)
    assert ex.tolist() == [[1, 3], [0, 1], [2, 4]]                 # ties go to the lower index
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-15)
    p = np.exp(lg.astype(np.float64))
    p /= p.sum(axis=1, keepdims=True)
    assert np.allclose(w[2], p[2, [2, 4]] / p[2, [2, 4]].sum(), rtol=1e-14)
    ex1, w1 = oracle.router(lg[:, :1], 1)
    assert ex1.tolist() == [[0], [0], [0]] and np.array_equal(w1, np.ones((3, 1)))


def _tiny_moe(E=4, B=3):
    mo = si.moe_layer(3, 32, 48, E, si.BF16, 16, B)
    for p in mo["experts"]:
        p.update(m1=None, tau1=0.0, bgu_fused=None, m2=None, tau2=0.0, bd_fused=None)
    return mo


def test_moe_tau_zero_is_dense_top2_moe_and_single_expert_is_glu():
    mo = _tiny_moe()
    dt = mo["dt"]
    hf = si.to_f32(mo["h"], dt)
    y, ex, w = oracle.moe_ffn(hf, mo["logits"], mo["experts"], dt, 2)
    F = mo["F"]
    want = np.zeros_like(y)
    p = np.exp(mo["logits"].astype(np.float64))
    p /= p.sum(axis=1, keepdims=True)
    for b in range(hf.shape[0]):
        top = np.argsort(-p[b], kind="stable")[:2]
        assert sorted(top.tolist()) == sorted(ex[b].tolist())
        for e in top:
            Wgu = si.to_f32(mo["experts"][e]["Wgu"], dt).astype(np.float64)
            Wd = si.to_f32(mo["experts"][e]["Wd"], dt).astype(np.float64)
            gu = hf[b].astype(np.float64) @ Wgu
            z = (gu[F:] * (gu[:F] / (1 + np.exp(-gu[:F])))).astype(np.float32).astype(np.float64)
            want[b] += p[b, e] / p[b, top].sum() * (z @ Wd)
    assert rel_l2(y, want) < 1e-13
    one = _tiny_moe(E=1)
    y1, _, _ = oracle.moe_ffn(si.to_f32(one["h"], dt), one["logits"], one["experts"], dt, 1)
    e0 = one["experts"][0]
    yg, _ = oracle.glu_ffn(si.to_f32(one["h"], dt), e0["Wgu"], e0["Wd"], dt, None, 0.0, None, None, 0.0, None)
    assert np.array_equal(y1, yg)


# ------------------------------------------------------------------ FFN sparsity accounting (Tables 5-6)

def test_ffn_sparsity_reproduces_printed_rows():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "ffn_sparsity_rows.txt")) if ln.strip() and ln[0] != "#"]
    assert len(rows) >= 30
    for _, up, gate, down, ffn in rows:
        got = oracle.ffn_sparsity(float(up), float(gate), float(down))
        assert abs(got - float(ffn)) <= 0.1 + 1e-9, (up, gate, down, ffn, got)
    # the shared-input form printed in Appendix B: 2/3 s_x + 1/3 s_gated
    assert abs(oracle.ffn_sparsity(42.0, 42.0, 61.7) - (2 / 3 * 42.0 + 1 / 3 * 61.7)) < 1e-12


# ---------------------------------------------------------------- mean / median estimators, scalar eta (Section 3)

def test_mean_and_median_agree_with_library_routines_and_closed_forms():
    rng = np.random.default_rng(7)
    for T, K in ((1, 3), (2, 5), (101, 7), (256, 4)):
        x = rng.standard_normal((T, K)).astype(np.float32)
        x[:, 0] = 1.5                                              # constant channel
        mean = oracle.mode_estimate(x, oracle.MEAN)
        med = oracle.mode_estimate(x, oracle.MEDIAN)
        # library mean differs from the in-order sum by rounding order only: one ulp of binary32 at most
        ref_mean = x.astype(np.float64).mean(axis=0)
        assert np.all(np.abs(mean - ref_mean) <= np.spacing(np.abs(ref_mean).astype(np.float32)))
        assert np.array_equal(med, np.median(x.astype(np.float64), axis=0).astype(np.float32))
        assert mean[0] == np.float32(1.5) and med[0] == np.float32(1.5)
    # closed forms: arithmetic progression (mean = median = midpoint), exact in binary64
    x = np.arange(1, 1001, dtype=np.float32).reshape(-1, 1)[::-1].copy()
    assert oracle.mode_estimate(x, oracle.MEAN)[0] == np.float32(500.5)
    assert oracle.mode_estimate(x, oracle.MEDIAN)[0] == np.float32(500.5)
    # odd count: the middle element itself; even: the mean of the two middle ones
    assert oracle.mode_estimate(np.float32([[5], [1], [9]]), oracle.MEDIAN)[0] == np.float32(5)
    assert oracle.mode_estimate(np.float32([[5], [1], [9], [6]]), oracle.MEDIAN)[0] == np.float32(5.5)


def test_mean_is_a_sum_in_row_order_in_binary64():
    # 2^20 + 2^-30 is exact in binary64 (50 bits apart) but not in binary32: the accumulator is binary64
    x = np.float32([[2.0 ** 20], [2.0 ** -30], [-(2.0 ** 20)]])
    assert oracle.mode_estimate(x, oracle.MEAN)[0] == np.float32((2.0 ** -30) / 3.0)
    # ... and rows are added in order: here the small term is absorbed before the large ones cancel
    x = np.float32([[2.0 ** 60], [2.0 ** -30], [-(2.0 ** 60)]])   # absorbed: 2^60 + 2^-30 == 2^60 in binary64
    assert oracle.mode_estimate(x, oracle.MEAN)[0] == np.float32(0.0)


def test_signed_zero_results_are_returned_as_plus_zero():
    x = np.float32([[-0.0], [-0.0]])
    for est in (oracle.MEAN, oracle.MEDIAN):
        m = oracle.mode_estimate(x, est)
        assert m[0] == 0 and not np.signbit(m[0])


def test_scalar_eta_pools_the_whole_tensor_and_is_broadcast():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal((64, 9)) + np.linspace(-2, 2, 9)[None, :]).astype(np.float32)
    for est in (oracle.HISTOGRAM, oracle.MEAN, oracle.MEDIAN):
        m = oracle.mode_estimate(x, est, oracle.SCALAR, nbins=32)
        assert m.shape == (9,) and np.all(m == m[0])
    eta_mean = oracle.mode_estimate(x, oracle.MEAN, oracle.SCALAR)[0]
    ref = x.astype(np.float64).mean()
    assert abs(eta_mean - ref) <= np.spacing(np.float32(abs(ref)))
    assert oracle.mode_estimate(x, oracle.MEDIAN, oracle.SCALAR)[0] == np.float32(np.median(x.astype(np.float64)))
    # pooled histogram mode == per-channel definition on the flattened tensor
    flat = x.reshape(-1, 1)
    assert oracle.mode_estimate(x, oracle.HISTOGRAM, oracle.SCALAR, nbins=32)[0] == oracle.mode(flat, 32)[0]
    # one channel: scalar and per-channel coincide
    one = x[:, :1].copy()
    for est in (oracle.HISTOGRAM, oracle.MEAN, oracle.MEDIAN):
        assert np.array_equal(oracle.mode_estimate(one, est, oracle.SCALAR, 32), oracle.mode_estimate(one, est, oracle.PER_CHANNEL, 32))


def test_kde_peak_agrees_with_the_library_kde_and_hand_cases():
    from scipy.stats import gaussian_kde
    rng = np.random.default_rng(23)
    T, K, G = 300, 5, 129
    x = np.stack([rng.normal(0.3, 1.0, T), rng.gamma(2.0, 1.0, T), rng.laplace(-1.0, 0.4, T),
                  np.abs(rng.normal(0, 1, T)) ** 1.5, rng.uniform(-1, 1, T) ** 3], axis=1).astype(np.float32)
    m = oracle.mode_estimate(x, oracle.KDE, oracle.PER_CHANNEL, G)
    for k in range(K):
        col = x[:, k].astype(np.float64)
        grid = col.min() + np.arange(G) * ((col.max() - col.min()) / (G - 1))
        lib_dens = gaussian_kde(col).evaluate(grid)        # Scott's factor T^(-1/5), covariance with divisor T - 1
        assert m[k] == np.float32(grid[int(np.argmax(lib_dens))])
        dens, g2 = oracle.kde_density(x, k, G)
        assert np.array_equal(g2, grid)
        norm = len(col) * np.std(col, ddof=1) * len(col) ** -0.2 * np.sqrt(2 * np.pi)
        assert np.allclose(dens / norm, lib_dens, rtol=1e-9, atol=0)
    # hand cases: a constant channel; a symmetric sample peaks at its centre; three of four points at the low end
    h = np.array([[0.75, -2.0, 1.0], [0.75, -1.0, 1.0], [0.75, 0.0, 1.0], [0.75, 0.0, 9.0],
                  [0.75, 0.0, 1.0], [0.75, 1.0, 1.0], [0.75, 2.0, 1.0]], np.float32)
    mh = oracle.mode_estimate(h, oracle.KDE, oracle.PER_CHANNEL, 5)
    assert mh[0] == np.float32(0.75) and mh[1] == np.float32(0.0) and mh[2] == np.float32(1.0)
    # translation by an exactly representable amount moves the peak by that amount
    assert np.array_equal(oracle.mode_estimate(h + np.float32(4.0), oracle.KDE, oracle.PER_CHANNEL, 5), mh + np.float32(4.0))


def test_estimators_rank_as_expected_on_a_skewed_distribution():
    # exponential-like (GELU-output-like) data: mode < median < mean; centring by a better mode estimate prunes more at fixed tau
    rng = np.random.default_rng(3)
    x = rng.exponential(1.0, size=(4096, 2)).astype(np.float32)
    hist = oracle.mode_estimate(x, oracle.HISTOGRAM, nbins=64)
    med = oracle.mode_estimate(x, oracle.MEDIAN)
    mean = oracle.mode_estimate(x, oracle.MEAN)
    assert np.all(hist < med) and np.all(med < mean)
    assert np.all(np.abs(med - math.log(2.0)) < 0.05) and np.all(np.abs(mean - 1.0) < 0.05)
    tau = np.float32(0.25)
    frac = [float(np.mean(np.abs(x - m[None, :]) < tau)) for m in (hist, med, mean)]
    assert frac[0] > frac[1] > frac[2]


# ---------------------------------------------------------------- non-GLU FFN (up -> GELU -> sparse down)

def _gelu64(v):
    return np.array([0.5 * t * (1.0 + math.erf(t / math.sqrt(2.0))) for t in np.ravel(v)]).reshape(np.shape(v))


def test_gelu_ffn_tau_zero_is_the_dense_mlp_and_gelu_has_its_textbook_values():
    g = si.glu_block(2, 48, 40, si.BF16, 8, 3)
    Wu = g["Wgu"][:, :40].copy()                                   # any [D, F] weight will do
    h = si.to_f32(g["h"], si.BF16)
    bu = np.linspace(-0.5, 0.5, 40).astype(np.float32)
    y, z = oracle.gelu_ffn(h, Wu, g["Wd"], si.BF16, None, 0.0, bu, None, 0.0, None)
    Wuf, Wdf = si.to_f32(Wu, si.BF16).astype(np.float64), si.to_f32(g["Wd"], si.BF16).astype(np.float64)
    u = h.astype(np.float64) @ Wuf + bu
    z_ref = _gelu64(u)
    assert np.allclose(z, z_ref, rtol=1e-6, atol=1e-9)
    assert np.allclose(y, z.astype(np.float64) @ Wdf, rtol=1e-12, atol=1e-12)
    # textbook values of the exact GELU through the same code path: one-channel "network" with unit weights
    one = si.to_bits(np.ones((1, 1)), si.BF16)
    for v, want in ((0.0, 0.0), (1.0, 0.8413447460685429), (-1.0, -0.15865525393145707), (6.0, 5.999999994080277), (-6.0, -5.919723e-09)):
        _, zz = oracle.gelu_ffn(np.float32([[v]]), one, one, si.BF16, None, 0.0, None, None, 0.0, None)
        assert abs(float(zz[0, 0]) - want) <= 1e-6 * max(1.0, abs(want)) + 1e-12


def test_gelu_ffn_is_the_composition_of_its_stages_and_honours_teacher_forcing():
    g = si.glu_block(2, 64, 56, si.BF16, 32, 2)
    Wu = g["Wgu"][:, 56:].copy()
    h = si.to_f32(g["h"], si.BF16)
    hc = si.to_f32(g["h_calib"], si.BF16)
    m1, tau1 = oracle.calibrate(hc, 0.3, 64)
    b1 = oracle.fold_bias(Wu, si.BF16, m1, None)
    _, zc = oracle.gelu_ffn(hc, Wu, g["Wd"], si.BF16, m1, tau1, b1, None, 0.0, None)
    m2, tau2 = oracle.calibrate(zc, 0.6, 64)
    b2 = oracle.fold_bias(g["Wd"], si.BF16, m2, None)
    y, z = oracle.gelu_ffn(h, Wu, g["Wd"], si.BF16, m1, tau1, b1, m2, tau2, b2)
    u = oracle.sparse_fc(h, Wu, si.BF16, m1, tau1, b1)
    assert np.array_equal(z, _gelu64(u).astype(np.float32))
    assert np.array_equal(y, oracle.sparse_fc(z, g["Wd"], si.BF16, m2, tau2, b2))
    z2 = z + np.float32(0.25)
    y2, z2o = oracle.gelu_ffn(h, Wu, g["Wd"], si.BF16, m1, tau1, b1, m2, tau2, b2, z_in=z2)
    assert np.array_equal(z2o, z2) and np.array_equal(y2, oracle.sparse_fc(z2, g["Wd"], si.BF16, m2, tau2, b2))
    # GELU output is skewed (bounded below near -0.17): the centred threshold prunes the target, the uncentred one less
    kept_c = float(np.mean(np.abs(zc - m2[None, :]) >= tau2))
    assert abs(kept_c - 0.4) < 0.02


# ---------------------------------------------------------------- 8-bit weights

def test_q8_oracle_reduces_to_the_16_bit_oracle_when_the_products_are_representable():
    # scale a power of two and |q| <= 127: scale * q is exact in fp16, so both oracles see the same real matrix
    rng = np.random.default_rng(5)
    K, N, B = 96, 24, 3
    q = rng.integers(-127, 128, size=(K, N)).astype(np.int8)
    scale = (2.0 ** rng.integers(-9, -5, size=K)).astype(np.float32)
    W16 = si.to_bits(scale[:, None].astype(np.float64) * q.astype(np.float64), si.F16)
    assert np.array_equal(si.to_f32(W16, si.F16), scale[:, None] * q.astype(np.float32))
    d = si.laplace_fc(4, K, N, si.F16, 8, B)
    xf = si.to_f32(d["x"], si.F16)
    m, bf = d["m_true"], np.linspace(-1, 1, N).astype(np.float32)
    for tau in (0.0, 0.2, 5.0):
        assert np.array_equal(oracle.sparse_fc_q8(xf, q, scale, m, tau, bf), oracle.sparse_fc(xf, W16, si.F16, m, tau, bf))
    assert np.array_equal(oracle.fold_bias_q8(q, scale, m, None), oracle.fold_bias(W16, si.F16, m, None))


def test_q8_brute_force_on_a_tiny_case_and_quantiser_properties():
    q = np.int8([[1, -2], [3, 4], [-128 + 1, 127]])
    scale = np.float32([0.5, 0.25, 2.0])
    x = np.float32([[1.0, -3.0, 0.1]])
    y = oracle.sparse_fc_q8(x, q, scale, None, 0.5, np.float32([10, 20]))
    assert np.array_equal(y, [[10 + 1.0 * 0.5 * 1 - 3.0 * 0.25 * 3, 20 + 1.0 * 0.5 * -2 - 3.0 * 0.25 * 4]])  # channel 2 pruned
    W = si.weight(4, 64, 40, si.BF16)
    qq, ss = si.quantise_q8(W, si.BF16)
    Wf = si.to_f32(W, si.BF16)
    assert qq.dtype == np.int8 and np.abs(qq).max() == 127 and np.all(np.abs(qq).max(axis=1) == 127)
    assert np.all(np.abs(ss[:, None] * qq - Wf) <= 0.5 * ss[:, None] * (1 + 1e-3))


# ---------------------------------------------------------------- group-wise 4-bit weights

def _pack_q4(q):
    return (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8)


def test_q4_oracle_reduces_to_the_16_bit_oracle_when_the_weights_are_representable():
    # scale a power of two, q - zero in -15..15: scale * (q - zero) is exact in bf16, so both oracles see one real matrix
    rng = np.random.default_rng(11)
    K, N, B, group = 80, 24, 3, 32      # 2.5 groups: the last one is short
    G = (K + group - 1) // group
    q = rng.integers(0, 16, size=(K, N)).astype(np.uint8)
    zero = rng.integers(0, 16, size=(G, N)).astype(np.uint8)
    scale = (2.0 ** rng.integers(-9, -5, size=(G, N))).astype(np.float32)
    gi = np.arange(K) // group
    Wreal = scale[gi].astype(np.float64) * (q.astype(np.float64) - zero[gi].astype(np.float64))
    W16 = si.to_bits(Wreal, si.BF16)
    assert np.array_equal(si.to_f32(W16, si.BF16).astype(np.float64), Wreal)
    d = si.laplace_fc(4, K, N, si.BF16, 8, B)
    xf = si.to_f32(d["x"], si.BF16)
    m, bf = d["m_true"], np.linspace(-1, 1, N).astype(np.float32)
    for tau in (0.0, 0.2, 5.0):
        assert np.array_equal(oracle.sparse_fc_q4(xf, _pack_q4(q), scale, zero, group, m, tau, bf),
                              oracle.sparse_fc(xf, W16, si.BF16, m, tau, bf))
    assert np.array_equal(oracle.fold_bias_q4(_pack_q4(q), scale, zero, group, m, None), oracle.fold_bias(W16, si.BF16, m, None))


def test_q4_hand_case_pins_the_nibble_order_the_group_index_and_the_zero_point():
    # K = 3 channels, group = 2 (channels 0, 1 | channel 2), N = 2 columns: one byte per row
    q = np.uint8([[1, 14], [5, 2], [9, 7]])           # (column 0, column 1) per row
    packed = np.uint8([[1 | (14 << 4)], [5 | (2 << 4)], [9 | (7 << 4)]])
    assert np.array_equal(_pack_q4(q), packed)
    scale = np.float32([[0.5, 0.25], [2.0, 4.0]])     # [group, column]
    zero = np.uint8([[3, 8], [1, 15]])
    x = np.float32([[1.0, -3.0, 2.0]])
    # W = scale * (q - zero): row 0: 0.5 * -2, 0.25 * 6; row 1: 0.5 * 2, 0.25 * -6; row 2 (group 1): 2 * 8, 4 * -8
    W = np.float64([[-1.0, 1.5], [1.0, -1.5], [16.0, -32.0]])
    y = oracle.sparse_fc_q4(x, packed, scale, zero, 2, None, 0.0, np.float32([10, 20]))
    assert np.array_equal(y, [[10 + 1.0 * W[0, 0] - 3.0 * W[1, 0] + 2.0 * W[2, 0], 20 + 1.0 * W[0, 1] - 3.0 * W[1, 1] + 2.0 * W[2, 1]]])
    y = oracle.sparse_fc_q4(x, packed, scale, zero, 2, None, 1.5, None)     # channel 0 pruned (|1| < 1.5)
    assert np.array_equal(y, [[-3.0 * W[1, 0] + 2.0 * W[2, 0], -3.0 * W[1, 1] + 2.0 * W[2, 1]]])
    m = np.float32([0.5, 0.0, -1.0])
    assert np.array_equal(oracle.fold_bias_q4(packed, scale, zero, 2, m, np.float32([1, 2])),
                          [1 + 0.5 * W[0, 0] - 1.0 * W[2, 0], 2 + 0.5 * W[0, 1] - 1.0 * W[2, 1]])


def test_q4_quantiser_properties():
    W = si.weight(4, 200, 24, si.BF16)
    packed, scale, zero = si.quantise_q4(W, si.BF16, 64)
    Wf = si.to_f32(W, si.BF16).astype(np.float64)
    q = np.empty((200, 24), np.int64)
    q[:, 0::2], q[:, 1::2] = packed & 15, packed >> 4
    gi = np.arange(200) // 64
    back = scale[gi].astype(np.float64) * (q - zero[gi].astype(np.int64))
    assert packed.shape == (200, 12) and scale.shape == (4, 24) and zero.shape == (4, 24) and q.min() >= 0 and q.max() == 15
    assert np.all(np.abs(back - Wf) <= scale[gi] * (1.0 + 1e-6))      # within one step (zero-point rounding adds up to half a step)


# ---------------------------------------------------------------- input recipe with overlapping sparsity (Appendix C)

def test_overlapping_rows_keep_the_union_sparse():
    """The recipe behind the test above: with full overlap the union over a context's rows stays near the per-row kept
    fraction, with none it grows like independent draws (CPU check of the generator through the oracle's mask)."""
    K = 4096
    fr = {}
    for ov in (0.0, 1.0):
        d = si.context_batch(4, K, 8, si.BF16, 64, 8, 1, ov, weights=False)
        xf = si.to_f32(d["x"], si.BF16)
        tau = oracle.tau(si.to_f32(d["x_calib"], si.BF16), d["m_true"], 0.6)
        keep, U, idx = oracle.mask(xf, d["m_true"], tau)
        fr[ov] = (keep.mean(), idx.size / K)
    assert abs(fr[0.0][0] - 0.4) < 0.05 and abs(fr[1.0][0] - 0.4) < 0.05
    assert fr[1.0][1] < 0.55 and fr[0.0][1] > 0.8
