"""Seeded synthetic inputs for the SCAP sparse-FC path.

This module only manufactures test data: storage-dtype bit patterns for weights,
activations, calibration sets and router logits.  It contains none of the
method's arithmetic (no thresholding, no centring, no FC, no quantile) and is
the one module that both the CPU oracle's callers and the CUDA path's callers
import, so that the two sides read byte-identical inputs.

Random numbers come from one counter-based generator, the published SplitMix64
finaliser applied to ``seed + (i+1) * golden_gamma``: element ``i`` of a stream
depends only on ``(seed, i)``, so any chunking or threading yields the same
arrays.  Normals are Box-Muller in float64, Laplace variates use the inverse
CDF.  Values are rounded once, round-to-nearest-even, to the storage dtype
(fp16 or bf16), and the resulting 16-bit patterns are what every consumer sees.

The activations of real checkpoints (Llama-2-7B, Mixtral-8x7B) and the C4
calibration slices the paper uses are not available offline; the recipes below
stand in for them with the same tensor shapes and with value distributions
chosen to exercise a non-zero per-channel mode.
"""
from __future__ import annotations

import concurrent.futures as _cf
import os as _os

import numpy as np

F16 = 0
BF16 = 1

SEED_BASE = 24120717400
# stream ids within a config
S_W, S_B, S_MODE, S_XCALIB, S_XTEST, S_LOGITS, S_GAMMA, S_W2, S_AUX = 0, 1, 2, 3, 4, 5, 6, 7, 8
EXPERT_STRIDE = 16

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 18


def stream_seed(config: int, stream: int, expert: int = 0) -> int:
    return SEED_BASE + 1000 * config + stream + EXPERT_STRIDE * expert


def _splitmix(seed: int, ctr: np.ndarray) -> np.ndarray:
    """SplitMix64 output number ``ctr`` (0-based) of the stream started at ``seed``."""
    with np.errstate(over="ignore"):
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + (ctr + np.uint64(1)) * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def _u01(seed: int, ctr: np.ndarray) -> np.ndarray:
    """Uniform on the open interval (0, 1): 53 random bits, centred in their cell."""
    return ((_splitmix(seed, ctr) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _chunks(n: int):
    for lo in range(0, n, _CHUNK):
        yield lo, min(n, lo + _CHUNK)


def _parallel_fill(n: int, fn, out: np.ndarray) -> np.ndarray:
    """out[lo:hi] = fn(lo, hi) over fixed chunks, on a small thread pool (numpy releases the GIL)."""
    spans = list(_chunks(n))
    if len(spans) <= 4:
        for lo, hi in spans:
            out[lo:hi] = fn(lo, hi)
        return out
    workers = max(1, min(16, (_os.cpu_count() or 1)))

    def run(span):
        lo, hi = span
        out[lo:hi] = fn(lo, hi)

    with _cf.ThreadPoolExecutor(workers) as ex:
        list(ex.map(run, spans))
    return out


def uniform(seed: int, n: int, lo: float = 0.0, hi: float = 1.0) -> np.ndarray:
    out = np.empty(n, np.float64)

    def fn(a, b):
        return lo + (hi - lo) * _u01(seed, np.arange(a, b, dtype=np.uint64))

    return _parallel_fill(n, fn, out)


def normal(seed: int, n: int) -> np.ndarray:
    """Standard normals; element i uses counters 2i and 2i+1 (Box-Muller, cosine branch)."""
    out = np.empty(n, np.float64)

    def fn(a, b):
        i = np.arange(a, b, dtype=np.uint64)
        u1 = _u01(seed, i * np.uint64(2))
        u2 = _u01(seed, i * np.uint64(2) + np.uint64(1))
        return np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * np.pi) * u2)

    return _parallel_fill(n, fn, out)


def laplace(seed: int, n: int, scale: float) -> np.ndarray:
    """Laplace(0, scale) by inverse CDF: v ~ U(-1/2, 1/2), L = -scale * sgn(v) * ln(1 - 2|v|)."""
    out = np.empty(n, np.float64)

    def fn(a, b):
        v = _u01(seed, np.arange(a, b, dtype=np.uint64)) - 0.5
        return -scale * np.sign(v) * np.log1p(-2.0 * np.abs(v))

    return _parallel_fill(n, fn, out)


# ---------------------------------------------------------------------------
# storage dtypes: 16-bit patterns
# ---------------------------------------------------------------------------

def to_bits(v: np.ndarray, dt: int) -> np.ndarray:
    """Round float64 values once (round-to-nearest-even) to fp16 / bf16; return the uint16 patterns."""
    if dt == F16:
        return np.asarray(v, np.float64).astype(np.float16).view(np.uint16)
    if dt != BF16:
        raise ValueError("dtype must be F16 or BF16")
    # bf16 keeps 8 significant bits.  Rounding the double straight to 8 bits (instead of going
    # through float32 first) avoids a double rounding.  frexp gives v = mant * 2^ex, |mant| in [0.5, 1).
    d = np.ascontiguousarray(v, np.float64)
    mant, ex = np.frexp(d)
    ex = np.maximum(ex, -125)                         # below 2^-126 the spacing stays 2^-133 (subnormals)
    q = np.ldexp(np.rint(np.ldexp(d, 8 - ex)), ex - 8)  # rint is round-half-even; ldexp is exact here
    f32 = q.astype(np.float32)                        # exact: q has at most 8 significant bits
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(d.shape)


def to_f32(bits: np.ndarray, dt: int) -> np.ndarray:
    """Exact widening of fp16 / bf16 bit patterns to float32."""
    bits = np.asarray(bits, np.uint16)
    if dt == F16:
        return bits.view(np.float16).astype(np.float32)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_torch(bits: np.ndarray, dt: int):
    """View uint16 patterns as a torch fp16 / bf16 CPU tensor (no copy, no rounding)."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.float16 if dt == F16 else torch.bfloat16)


# ---------------------------------------------------------------------------
# recipes
# ---------------------------------------------------------------------------

def weight(config: int, K: int, N: int, dt: int, stream: int = S_W, expert: int = 0, std: float = 0.02) -> np.ndarray:
    """W[K, N] ~ N(0, std^2), input-channel-major (row k holds every output of input channel k)."""
    seed = stream_seed(config, stream, expert)
    out = np.empty(K * N, np.uint16)

    def fn(a, b):
        i = np.arange(a, b, dtype=np.uint64)
        u1 = _u01(seed, i * np.uint64(2))
        u2 = _u01(seed, i * np.uint64(2) + np.uint64(1))
        return to_bits(std * (np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * np.pi) * u2)), dt)

    return _parallel_fill(K * N, fn, out).reshape(K, N)


def laplace_fc(config: int, K: int, N: int, dt: int, T_calib: int, B: int, with_bias: bool = True,
               scale: float = 0.3) -> dict:
    """Single FC with Laplace-around-a-mode inputs: m_k ~ U(-0.5, 0.5), x_k = m_k + Laplace(0, scale)."""
    m_true = uniform(stream_seed(config, S_MODE), K, -0.5, 0.5)
    xc = m_true[None, :] + laplace(stream_seed(config, S_XCALIB), T_calib * K, scale).reshape(T_calib, K)
    xt = m_true[None, :] + laplace(stream_seed(config, S_XTEST), B * K, scale).reshape(B, K)
    d = {
        "dt": dt, "K": K, "N": N,
        "W": weight(config, K, N, dt),
        "m_true": m_true.astype(np.float32),
        "x_calib": to_bits(xc, dt),
        "x": to_bits(xt, dt),
        "laplace_scale": scale,
    }
    d["b"] = to_bits(0.01 * normal(stream_seed(config, S_B), N), dt) if with_bias else None
    return d


def context_batch(config: int, K: int, N: int, dt: int, T_calib: int, B: int, n_ctx: int, overlap: float,
                  active_frac: float = 0.5, hi: float = 0.3, lo: float = 0.01, weights: bool = True) -> dict:
    """Rows whose large activations fall on a per-context set of channels (Appendix C of the paper: the rows of one batch
    - beams of one prompt, tokens of one request - share part of their sparsity pattern).

    Every context c has an active set A_c (each channel with probability active_frac).  Row b belongs to context
    b mod n_ctx; channel k of row b is "on" if it is in A_c - with probability ``overlap`` per (row, channel) - or else
    by an independent draw with probability active_frac.  x[b,k] = m_k + Laplace(0, hi) where on, Laplace(0, lo)
    elsewhere.  overlap = 1: all rows of a context share one pattern; overlap = 0: the rows are independent.
    With the defaults and a 60 % sparsity target the threshold falls between the two populations: a row keeps about
    four fifths of its "on" channels and next to none of the others, so the union over a context's rows is bounded by
    the context's active set (half the channels) at overlap 1 and approaches all channels at overlap 0.
    The calibration rows are drawn the same way (context t mod n_ctx).  Returns also ``ctx`` [B]."""
    m_true = uniform(stream_seed(config, S_MODE), K, -0.5, 0.5)
    A = uniform(stream_seed(config, S_GAMMA), n_ctx * K).reshape(n_ctx, K) < active_frac

    def rows(stream, T):
        pick = uniform(stream_seed(config, stream, 1), T * K).reshape(T, K) < overlap
        own = uniform(stream_seed(config, stream, 2), T * K).reshape(T, K) < active_frac
        on = np.where(pick, A[np.arange(T) % n_ctx], own)
        noise = laplace(stream_seed(config, stream), T * K, 1.0).reshape(T, K)
        return m_true[None, :] + noise * np.where(on, hi, lo), on

    xc, _ = rows(S_XCALIB, T_calib)
    xt, on = rows(S_XTEST, B)
    d = {"dt": dt, "K": K, "N": N, "m_true": m_true.astype(np.float32), "x_calib": to_bits(xc, dt), "x": to_bits(xt, dt),
         "ctx": (np.arange(B) % n_ctx).astype(np.int32), "on": on, "b": None}
    if weights:
        d["W"] = weight(config, K, N, dt)
    return d


def _silu(g: np.ndarray) -> np.ndarray:
    return g / (1.0 + np.exp(-g))


def gated_activations(config: int, stream: int, T: int, K: int, dt: int) -> np.ndarray:
    """Rows of silu(g) * u with g, u ~ N(0,1) i.i.d.: the shape of a SwiGLU down-projection input."""
    gu = normal(stream_seed(config, stream), 2 * T * K).reshape(2, T, K)
    return to_bits(_silu(gu[0]) * gu[1], dt)


def down_proj(config: int, K: int, N: int, dt: int, T_calib: int, B: int) -> dict:
    """FFN down projection fed by silu(g)*u activations; no bias."""
    return {
        "dt": dt, "K": K, "N": N,
        "W": weight(config, K, N, dt),
        "b": None,
        "x_calib": gated_activations(config, S_XCALIB, T_calib, K, dt),
        "x": gated_activations(config, S_XTEST, B, K, dt),
    }


def glu_block(config: int, D: int, F: int, dt: int, T_calib: int, B: int, lognormal_sigma: float = 0.5,
              expert: int = 0, weights: bool = True) -> dict:
    """SwiGLU FFN block: h = gamma * N(0,1) with per-channel gamma ~ LogNormal(0, sigma).

    Wgu[D, 2F] holds gate (columns 0..F-1) and up (columns F..2F-1) of one input channel in one row;
    Wd[F, D].  sigma = 0 gives gamma = 1 (plain N(0,1) hidden states).
    """
    if lognormal_sigma > 0:
        gamma = np.exp(lognormal_sigma * normal(stream_seed(config, S_GAMMA, expert), D))
    else:
        gamma = np.ones(D)
    hc = gamma[None, :] * normal(stream_seed(config, S_XCALIB, expert), T_calib * D).reshape(T_calib, D)
    ht = gamma[None, :] * normal(stream_seed(config, S_XTEST, expert), B * D).reshape(B, D)
    d = {"dt": dt, "D": D, "F": F, "gamma": gamma, "h_calib": to_bits(hc, dt), "h": to_bits(ht, dt)}
    if weights:
        d["Wgu"] = weight(config, D, 2 * F, dt, S_W, expert)
        d["Wd"] = weight(config, F, D, dt, S_W2, expert)
    return d


def moe_layer(config: int, D: int, F: int, E: int, dt: int, T_calib: int, B: int) -> dict:
    """E experts of SwiGLU weights, N(0,1) hidden states, router logits ~ N(0,1).

    Each expert gets its own calibration stream of T_calib hidden states.
    """
    experts = []
    for e in range(E):
        experts.append({
            "Wgu": weight(config, D, 2 * F, dt, S_W, e),
            "Wd": weight(config, F, D, dt, S_W2, e),
            "h_calib": to_bits(normal(stream_seed(config, S_XCALIB, e), T_calib * D).reshape(T_calib, D), dt),
        })
    h = to_bits(normal(stream_seed(config, S_XTEST), B * D).reshape(B, D), dt)
    logits = normal(stream_seed(config, S_LOGITS), B * E).reshape(B, E).astype(np.float32)
    return {"dt": dt, "D": D, "F": F, "E": E, "experts": experts, "h": h, "logits": logits}


# The five published workload descriptions, at full size.  Tests pass smaller dimensions
# to the recipe functions above; bench and the full-size parity tests call these.

def config0(B: int = 1) -> dict:
    return laplace_fc(0, 1024, 1024, F16, 256, B)


def config1(B: int = 1) -> dict:
    return down_proj(1, 11008, 4096, BF16, 1024, B)


def config2(B: int = 1) -> dict:
    return glu_block(2, 4096, 11008, BF16, 1024, B)


def config3(B: int = 1) -> dict:
    return moe_layer(3, 4096, 14336, 8, BF16, 2048, B)


def config4_fc(K: int, N: int, B: int, T_calib: int = 2048) -> dict:
    return laplace_fc(4, K, N, BF16, T_calib, B, with_bias=False)


def quantise_q8(W_bits: np.ndarray, dt: int):
    """Symmetric 8-bit quantisation of a 16-bit weight, one scale per input channel (row): scale = max|row| / 127
    (1 for an all-zero row), q = round-half-even(W / scale) clipped to [-127, 127].  Returns (int8 [K,N], float32 [K])."""
    Wf = to_f32(W_bits, dt).astype(np.float64)
    amax = np.abs(Wf).max(axis=1)
    scale = np.where(amax > 0, amax / 127.0, 1.0).astype(np.float32)
    q = np.clip(np.rint(Wf / scale.astype(np.float64)[:, None]), -127, 127).astype(np.int8)
    return q, scale


def quantise_q4(W_bits: np.ndarray, dt: int, group: int = 128):
    """Asymmetric group-wise 4-bit quantisation of a 16-bit weight: for every group of ``group`` consecutive input channels
    (rows) and every output column, scale = (max - min) / 15 (1 where the group is constant), zero = round(-min / scale)
    clipped to 0..15, q = round(W / scale) + zero clipped to 0..15.  Returns (packed uint8 [K, N/2] with the even column in
    the low nibble, float32 scale [K/group, N], uint8 zero [K/group, N])."""
    Wf = to_f32(W_bits, dt).astype(np.float64)
    K, N = Wf.shape
    assert N % 2 == 0
    G = (K + group - 1) // group
    scale = np.empty((G, N), np.float32)
    zero = np.empty((G, N), np.uint8)
    q = np.empty((K, N), np.uint8)
    for g in range(G):
        blk = Wf[g * group:(g + 1) * group]
        lo, hi = blk.min(axis=0), blk.max(axis=0)
        sc = np.where(hi > lo, (hi - lo) / 15.0, 1.0).astype(np.float32)
        zp = np.clip(np.rint(-lo / sc.astype(np.float64)), 0, 15)
        scale[g], zero[g] = sc, zp.astype(np.uint8)
        q[g * group:(g + 1) * group] = np.clip(np.rint(blk / sc.astype(np.float64)[None, :]) + zp[None, :], 0, 15).astype(np.uint8)
    packed = (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8)
    return packed, scale, zero
