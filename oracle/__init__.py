"""Python face of the CPU oracle (TEST INFRASTRUCTURE ONLY).

Thin numpy/ctypes wrappers over ``scap_oracle.c`` plus the few compositions that are plainer
in numpy (the mixture-of-experts layer, a BLAS-backed batch evaluation of SwiGLU stage 1 used
only to manufacture calibration activations).  Nothing here is imported by the CUDA library
or its Python binding; only tests, the smoke check and the benchmark's CPU-baseline leg use it.

Every function cites the passage of the paper it follows; see the header of ``scap_oracle.c``
for the floating-point conventions and for the list of "parity unpinned" parts.
"""
from __future__ import annotations

import concurrent.futures as _cf
import ctypes as C
import os
import subprocess

import numpy as np

F16, BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "scap_oracle.c")
_LIB = os.path.join(_HERE, "libscap_oracle.so")

_CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-std=c99"]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fused multiply-add, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i, f, d = C.c_void_p, C.c_int, C.c_float, C.c_double
        L.scap_oracle_widen_array.argtypes = [vp, i, C.c_long, vp]
        L.scap_oracle_widen_array.restype = None
        L.scap_oracle_mask.argtypes = [vp, vp, f, i, i, vp, vp, vp, vp]
        L.scap_oracle_mask.restype = i
        L.scap_oracle_sparse_fc.argtypes = [vp, vp, i, vp, f, vp, i, i, i, vp]
        L.scap_oracle_sparse_fc.restype = None
        L.scap_oracle_sparse_fc_cols.argtypes = [vp, vp, i, vp, f, vp, i, i, i, i, i, vp]
        L.scap_oracle_sparse_fc_cols.restype = None
        L.scap_oracle_dense_fc.argtypes = [vp, vp, i, vp, i, i, i, vp]
        L.scap_oracle_dense_fc.restype = None
        L.scap_oracle_fold_bias.argtypes = [vp, i, vp, vp, i, i, vp]
        L.scap_oracle_fold_bias.restype = None
        L.scap_oracle_mode.argtypes = [vp, i, i, i, vp]
        L.scap_oracle_mode.restype = None
        L.scap_oracle_mean.argtypes = [vp, i, i, vp]
        L.scap_oracle_mean.restype = None
        L.scap_oracle_median.argtypes = [vp, i, i, vp]
        L.scap_oracle_median.restype = None
        L.scap_oracle_kde.argtypes = [vp, i, i, i, vp, i, vp]
        L.scap_oracle_kde.restype = None
        L.scap_oracle_eta_mean.argtypes = [vp, i, i]
        L.scap_oracle_eta_mean.restype = f
        L.scap_oracle_tau.argtypes = [vp, i, i, vp, d, vp, vp]
        L.scap_oracle_tau.restype = f
        L.scap_oracle_glu_ffn.argtypes = [vp, vp, vp, i, vp, f, vp, vp, f, vp, i, i, i, vp, vp, vp]
        L.scap_oracle_glu_ffn.restype = None
        L.scap_oracle_gelu_ffn.argtypes = [vp, vp, vp, i, vp, f, vp, vp, f, vp, i, i, i, vp, vp, vp]
        L.scap_oracle_gelu_ffn.restype = None
        L.scap_oracle_sparse_fc_q8.argtypes = [vp, vp, vp, vp, f, vp, i, i, i, vp]
        L.scap_oracle_sparse_fc_q8.restype = None
        L.scap_oracle_fold_bias_q8.argtypes = [vp, vp, vp, vp, i, i, vp]
        L.scap_oracle_fold_bias_q8.restype = None
        L.scap_oracle_sparse_fc_q4.argtypes = [vp, vp, vp, vp, i, vp, f, vp, i, i, i, vp]
        L.scap_oracle_sparse_fc_q4.restype = None
        L.scap_oracle_fold_bias_q4.argtypes = [vp, vp, vp, i, vp, vp, i, i, vp]
        L.scap_oracle_fold_bias_q4.restype = None
        L.scap_oracle_router.argtypes = [vp, i, i, i, vp, vp]
        L.scap_oracle_router.restype = None
        L.scap_oracle_ffn_sparsity.argtypes = [d, d, d]
        L.scap_oracle_ffn_sparsity.restype = d
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, np.float32)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "storage arrays are uint16 bit patterns"
    return a


def widen(bits: np.ndarray, dt: int) -> np.ndarray:
    """Exact fp16/bf16 -> binary32 widening done by the oracle's own routine."""
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float32)
    lib().scap_oracle_widen_array(_p(bits), dt, bits.size, _p(out))
    return out


def mask(xf, m, tau, want_d=False):
    """Eq. 2 / Alg. 3 centre + threshold.  Returns (keep[B,K] bool, U[K] bool, idx uint32[nnz])  (+ d[B,K])."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    m = _f32(m)
    keep = np.empty((B, K), np.uint8)
    U = np.empty(K, np.uint8)
    idx = np.empty(K, np.uint32)
    d = np.empty((B, K), np.float32) if want_d else None
    nnz = lib().scap_oracle_mask(_p(xf), _p(m), float(np.float32(tau)), B, K, _p(keep), _p(d), _p(U), _p(idx))
    out = (keep.astype(bool), U.astype(bool), idx[:nnz].copy())
    return out + (d,) if want_d else out


def sparse_fc(xf, W, dt, m, tau, b_fused, threads: int = 1, cols=None):
    """Eq. 3 / Alg. 3.  y[B,N] float64.  ``cols=(n0,n1)`` restricts to a column range;
    ``threads`` > 1 spreads disjoint column ranges over threads (each column's sum is unchanged)."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    W = _u16(W)
    assert W.shape[0] == K
    N = W.shape[1]
    m, b_fused = _f32(m), _f32(b_fused)
    tau = float(np.float32(tau))
    n0, n1 = (0, N) if cols is None else cols
    if threads <= 1:
        y = np.empty((B, n1 - n0), np.float64)
        lib().scap_oracle_sparse_fc_cols(_p(xf), _p(W), dt, _p(m), tau, _p(b_fused), B, K, N, n0, n1, _p(y))
        return y
    edges = np.linspace(n0, n1, threads + 1).astype(int)
    parts = [None] * threads

    def run(t):
        a, b = int(edges[t]), int(edges[t + 1])
        yy = np.empty((B, b - a), np.float64)
        if b > a:
            lib().scap_oracle_sparse_fc_cols(_p(xf), _p(W), dt, _p(m), tau, _p(b_fused), B, K, N, a, b, _p(yy))
        parts[t] = yy

    with _cf.ThreadPoolExecutor(threads) as ex:
        list(ex.map(run, range(threads)))
    return np.concatenate(parts, axis=1)


def sparse_fc_full(xf, W, dt, m, tau, b_fused):
    """The single-loop-nest form (no column ranges); the tests check it equals ``sparse_fc``."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    W = _u16(W)
    N = W.shape[1]
    y = np.empty((B, N), np.float64)
    lib().scap_oracle_sparse_fc(_p(xf), _p(W), dt, _p(_f32(m)), float(np.float32(tau)), _p(_f32(b_fused)),
                                B, K, N, _p(y))
    return y


def dense_fc(xf, W, dt, b):
    """Eq. 1: y = xW + b, float64."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    W = _u16(W)
    N = W.shape[1]
    y = np.empty((B, N), np.float64)
    lib().scap_oracle_dense_fc(_p(xf), _p(W), dt, _p(_f32(b)), B, K, N, _p(y))
    return y


def fold_bias(W, dt, m, b_bits):
    """Eq. 5-6: b_fused = b + mW, float64.  ``b_bits`` are storage-dtype patterns or None."""
    W = _u16(W)
    K, N = W.shape
    out = np.empty(N, np.float64)
    lib().scap_oracle_fold_bias(_p(W), dt, _p(_f32(m)), _p(None if b_bits is None else _u16(b_bits)), K, N, _p(out))
    return out


def mode(xf_calib, nbins: int = 2048):
    """Per-channel histogram arg-max mode estimate (Section 3), binary32."""
    xf = _f32(np.atleast_2d(xf_calib))
    T, K = xf.shape
    m = np.empty(K, np.float32)
    lib().scap_oracle_mode(_p(xf), T, K, nbins, _p(m))
    return m


HISTOGRAM, MEAN, MEDIAN, KDE = 0, 1, 2, 3   # mode estimators (Section 3, "Determination of mode value")
PER_CHANNEL, SCALAR = 0, 1             # one mode per input channel, or the paper's single eta per FC


def mode_estimate(xf_calib, estimator: int = HISTOGRAM, scope: int = PER_CHANNEL, nbins: int = 2048):
    """m[K] by the chosen estimator; with scope SCALAR the single eta of the pooled tensor, broadcast to K entries."""
    xf = _f32(np.atleast_2d(xf_calib))
    T, K = xf.shape
    if scope == PER_CHANNEL:
        if estimator == HISTOGRAM:
            return mode(xf, nbins)
        m = np.empty(K, np.float32)
        if estimator == KDE:
            lib().scap_oracle_kde(_p(xf), T, K, int(nbins), _p(m), -1, None)
            return m
        (lib().scap_oracle_mean if estimator == MEAN else lib().scap_oracle_median)(_p(xf), T, K, _p(m))
        return m
    if estimator == KDE:
        raise ValueError("the KDE peak is defined per channel only")
    if estimator == MEAN:
        eta = np.float32(lib().scap_oracle_eta_mean(_p(xf), T, K))
    else:
        flat = np.ascontiguousarray(xf.reshape(T * K, 1))
        one = np.empty(1, np.float32)
        if estimator == HISTOGRAM:
            lib().scap_oracle_mode(_p(flat), T * K, 1, nbins, _p(one))
        else:
            lib().scap_oracle_median(_p(flat), T * K, 1, _p(one))
        eta = one[0]
    return np.full(K, eta, np.float32)


def kde_density(xf_calib, k: int, G: int):
    """The G (unnormalised) densities of channel k on its grid, and the grid itself (binary64)."""
    xf = _f32(np.atleast_2d(xf_calib))
    T, K = xf.shape
    m = np.empty(K, np.float32)
    dens = np.empty(G, np.float64)
    lib().scap_oracle_kde(_p(xf), T, K, int(G), _p(m), int(k), dens.ctypes.data_as(C.c_void_p))
    lo, hi = np.float64(xf[:, k].min()), np.float64(xf[:, k].max())
    grid = lo + np.arange(G, dtype=np.float64) * ((hi - lo) / (G - 1))
    return dens, grid


def calibrate_ex(xf_calib, s: float, estimator: int = HISTOGRAM, scope: int = PER_CHANNEL, nbins: int = 2048):
    """Mode by the chosen estimator and scope, then the threshold on the centred importance."""
    xf = _f32(np.atleast_2d(xf_calib))
    m = mode_estimate(xf, estimator, scope, nbins)
    return m, tau(xf, m, s)


def tau(xf_calib, m, s: float, want_neighbours=False):
    """Eq. 2: tau = Quantile(|X_calib - m|, s), linear interpolation, pooled over all T*K values."""
    xf = _f32(np.atleast_2d(xf_calib))
    T, K = xf.shape
    vj, vj1 = C.c_float(0), C.c_float(0)
    t = lib().scap_oracle_tau(_p(xf), T, K, _p(_f32(m)), float(s), C.byref(vj), C.byref(vj1))
    t = np.float32(t)
    return (t, np.float32(vj.value), np.float32(vj1.value)) if want_neighbours else t


def calibrate(xf_calib, s: float, nbins: int = 2048):
    """Mode, then threshold on the centred importance (Section 3: the two run in sequence).
    nbins == 0 means no centring (m = 0)."""
    xf = _f32(np.atleast_2d(xf_calib))
    m = mode(xf, nbins) if nbins > 0 else np.zeros(xf.shape[1], np.float32)
    return m, tau(xf, m, s)


def sparse_fc_q8(xf, Wq, scale, m, tau, b_fused):
    """Sparse FC on 8-bit weights: W[k,n] = scale[k] * Wq[k,n] (signed 8-bit, one scale per input channel)."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    Wq = np.ascontiguousarray(Wq, np.int8)
    N = Wq.shape[1]
    y = np.empty((B, N), np.float64)
    lib().scap_oracle_sparse_fc_q8(_p(xf), _p(Wq), _p(_f32(scale)), _p(_f32(m)), float(np.float32(tau)), _p(_f32(b_fused)), B, K, N, _p(y))
    return y


def fold_bias_q8(Wq, scale, m, b):
    Wq = np.ascontiguousarray(Wq, np.int8)
    K, N = Wq.shape
    out = np.empty(N, np.float64)
    lib().scap_oracle_fold_bias_q8(_p(Wq), _p(_f32(scale)), _p(_f32(m)), _p(_f32(b)), K, N, _p(out))
    return out


def sparse_fc_q4(xf, Wq, scale, zero, group, m, tau, b_fused):
    """Eq. 2-3 on group-wise 4-bit weights: Wq[K, N/2] uint8 (two codes per byte, even column in the low nibble),
    scale[K/group, N] float32, zero[K/group, N] uint8; W = scale * (q - zero).  Returns y[B,N] float64."""
    xf = _f32(np.atleast_2d(xf))
    B, K = xf.shape
    Wq = np.ascontiguousarray(Wq, np.uint8)
    N = Wq.shape[1] * 2
    scale = _f32(scale)
    zero = np.ascontiguousarray(zero, np.uint8)
    G = (K + group - 1) // group
    assert Wq.shape == (K, N // 2) and scale.shape == (G, N) and zero.shape == (G, N)
    y = np.empty((B, N), np.float64)
    lib().scap_oracle_sparse_fc_q4(_p(xf), _p(Wq), _p(scale), _p(zero), int(group), _p(_f32(m)), float(np.float32(tau)),
                                   _p(_f32(b_fused)), B, K, N, _p(y))
    return y


def fold_bias_q4(Wq, scale, zero, group, m, b):
    """Eq. 5-6 on group-wise 4-bit weights: b + m W in float64."""
    Wq = np.ascontiguousarray(Wq, np.uint8)
    K, N = Wq.shape[0], Wq.shape[1] * 2
    out = np.empty(N, np.float64)
    lib().scap_oracle_fold_bias_q4(_p(Wq), _p(_f32(scale)), _p(np.ascontiguousarray(zero, np.uint8)), int(group), _p(_f32(m)),
                                   _p(_f32(b)), K, N, _p(out))
    return out


def glu_ffn(hf, Wgu, Wd, dt, m1, tau1, bgu_fused, m2, tau2, bd_fused, z_in=None):
    """Alg. 2 (SCAP SwiGLU).  Returns (y[B,D] float64, z32[B,F] float32)."""
    hf = _f32(np.atleast_2d(hf))
    B, D = hf.shape
    Wgu, Wd = _u16(Wgu), _u16(Wd)
    F = Wd.shape[0]
    assert Wgu.shape == (D, 2 * F) and Wd.shape == (F, D)
    y = np.empty((B, D), np.float64)
    z = np.empty((B, F), np.float32)
    zin = None if z_in is None else _f32(z_in)
    lib().scap_oracle_glu_ffn(_p(hf), _p(Wgu), _p(Wd), dt, _p(_f32(m1)), float(np.float32(tau1)), _p(_f32(bgu_fused)),
                              _p(_f32(m2)), float(np.float32(tau2)), _p(_f32(bd_fused)), B, D, F, _p(zin), _p(y), _p(z))
    return y, z


def gelu_ffn(hf, Wu, Wd, dt, m1, tau1, bu_fused, m2, tau2, bd_fused, z_in=None):
    """Non-GLU FFN (up -> exact GELU -> mode-centred sparse down).  Returns (y[B,D] float64, z32[B,F] float32)."""
    hf = _f32(np.atleast_2d(hf))
    B, D = hf.shape
    Wu, Wd = _u16(Wu), _u16(Wd)
    F = Wd.shape[0]
    assert Wu.shape == (D, F) and Wd.shape == (F, D)
    y = np.empty((B, D), np.float64)
    z = np.empty((B, F), np.float32)
    zin = None if z_in is None else _f32(z_in)
    lib().scap_oracle_gelu_ffn(_p(hf), _p(Wu), _p(Wd), dt, _p(_f32(m1)), float(np.float32(tau1)), _p(_f32(bu_fused)),
                               _p(_f32(m2)), float(np.float32(tau2)), _p(_f32(bd_fused)), B, D, F, _p(zin), _p(y), _p(z))
    return y, z


def glu_stage1_batch(hf, Wgu, dt, m1, tau1, bgu_fused):
    """z = up * silu(gate) for many rows at once, with a float64 library matmul as the FC step.

    Used only to manufacture stage-2 calibration activations (hundreds of tokens), where the
    plain loops would take minutes.  Same definition as the first half of ``glu_ffn``; the
    tests check the two agree to rounding on small inputs.  Returns z32[T,F] float32.
    """
    hf = _f32(np.atleast_2d(hf))
    keep, _, _, d = mask(hf, m1, tau1, want_d=True)
    m1v = np.zeros(hf.shape[1]) if m1 is None else np.asarray(m1, np.float64)
    xc = np.where(keep, hf.astype(np.float64) - m1v[None, :], 0.0)
    Wf = widen(Wgu, dt).astype(np.float64)
    gu = xc @ Wf
    if bgu_fused is not None:
        gu += np.asarray(bgu_fused, np.float64)[None, :]
    F = Wgu.shape[1] // 2
    g, u = gu[:, :F], gu[:, F:]
    return (u * (g / (1.0 + np.exp(-g)))).astype(np.float32)


def router(logits, top_k: int = 2):
    """softmax -> top-k (ties to the lower index) -> renormalise.  (experts[B,k] int32, weights[B,k] float64)"""
    lg = _f32(np.atleast_2d(logits))
    B, E = lg.shape
    ex = np.empty((B, top_k), np.int32)
    w = np.empty((B, top_k), np.float64)
    lib().scap_oracle_router(_p(lg), B, E, top_k, _p(ex), _p(w))
    return ex, w


def moe_ffn(hf, logits, experts, dt, top_k: int = 2):
    """Mixture-of-experts FFN: y[b] = sum over the row's selected experts of w_e * glu_ffn_e(h[b]).

    ``experts`` is a list of dicts with Wgu, Wd, m1, tau1, bgu_fused, m2, tau2, bd_fused.
    Rows are independent under per-element pruning, so each (row, expert) pair is evaluated alone.
    """
    hf = _f32(np.atleast_2d(hf))
    B, D = hf.shape
    ex, w = router(logits, top_k)
    y = np.zeros((B, D), np.float64)
    for b in range(B):
        for j in range(top_k):
            p = experts[int(ex[b, j])]
            yb, _ = glu_ffn(hf[b:b + 1], p["Wgu"], p["Wd"], dt, p["m1"], p["tau1"], p["bgu_fused"],
                            p["m2"], p["tau2"], p["bd_fused"])
            y[b] += w[b, j] * yb[0]
    return y, ex, w


def ffn_sparsity(s_up, s_gate, s_down):
    return lib().scap_oracle_ffn_sparsity(float(s_up), float(s_gate), float(s_down))
