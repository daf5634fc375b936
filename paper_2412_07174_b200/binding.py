"""ctypes binding of libscap_b200.so: same names as the C ABI, marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import torch

__all__ = [
    "SCAP_F16", "SCAP_BF16", "ScapError", "lib", "lib_path", "status_string", "scap_version", "scap_tune", "scap_device_status",
    "scap_calibrate_workspace", "scap_calibrate", "scap_calibrate_ex", "SCAP_MODE_HISTOGRAM", "SCAP_MODE_MEAN", "SCAP_MODE_MEDIAN", "SCAP_MODE_KDE",
    "SCAP_ETA_PER_CHANNEL", "SCAP_ETA_SCALAR", "scap_fold_bias_workspace", "scap_fold_bias",
    "scap_fc_workspace", "scap_sparse_fc", "scap_dense_fc", "scap_sparse_fc_q8", "scap_dense_fc_q8", "scap_fold_bias_q8",
    "scap_sparse_fc_q4", "scap_dense_fc_q4", "scap_fold_bias_q4", "scap_grouped_workspace", "scap_sparse_fc_grouped",
    "scap_fc_host_workspace", "scap_sparse_fc_host",
    "scap_glu_workspace", "scap_glu_ffn", "scap_gelu_ffn_workspace", "scap_gelu_ffn", "scap_glu_static_capacity", "scap_glu_ffn_static", "scap_moe_workspace",
    "scap_moe_ffn", "ScapExpert", "dtype_of", "EXPORTS",
]

SCAP_F16, SCAP_BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))

# every symbol include/scap.h declares
EXPORTS = [
    "scap_status_string", "scap_version", "scap_tune", "scap_device_status", "scap_calibrate_workspace", "scap_calibrate",
    "scap_calibrate_ex", "scap_fold_bias_workspace", "scap_fold_bias", "scap_fc_workspace", "scap_sparse_fc", "scap_dense_fc",
    "scap_sparse_fc_q8", "scap_dense_fc_q8", "scap_fold_bias_q8", "scap_sparse_fc_q4", "scap_dense_fc_q4", "scap_fold_bias_q4",
    "scap_grouped_workspace", "scap_sparse_fc_grouped", "scap_fc_host_workspace", "scap_sparse_fc_host", "scap_glu_workspace", "scap_glu_ffn", "scap_gelu_ffn_workspace",
    "scap_gelu_ffn", "scap_glu_static_capacity", "scap_glu_ffn_static", "scap_moe_workspace", "scap_moe_ffn",
]


class ScapError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s" % (where, status_string(code)))


class ScapExpert(C.Structure):
    """Mirror of ``scap_expert``: device pointers of one expert's weights and calibration."""
    _fields_ = [(n, C.c_void_p) for n in ("Wgu", "Wd", "m1", "tau1", "bgu_fused", "m2", "tau2", "bd_fused")]


def lib_path() -> str:
    return os.path.join(_HERE, "libscap_b200.so")


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError("%s is missing: run `python -m paper_2412_07174_b200.build` (needs nvcc)" % path)
    L = C.CDLL(path)
    vp, i, sz, d = C.c_void_p, C.c_int, C.c_size_t, C.c_double
    L.scap_status_string.argtypes = [i]
    L.scap_status_string.restype = C.c_char_p
    L.scap_version.argtypes = []
    L.scap_version.restype = i
    L.scap_tune.argtypes = [C.c_char_p, i]
    L.scap_tune.restype = i
    L.scap_device_status.argtypes = []
    L.scap_device_status.restype = i
    L.scap_calibrate_workspace.argtypes = [i, i, i]
    L.scap_calibrate_workspace.restype = sz
    L.scap_calibrate.argtypes = [vp, i, i, i, d, i, vp, vp, vp, sz, vp]
    L.scap_calibrate.restype = i
    L.scap_calibrate_ex.argtypes = [vp, i, i, i, d, i, i, i, vp, vp, vp, sz, vp]
    L.scap_calibrate_ex.restype = i
    L.scap_fold_bias_workspace.argtypes = [i, i]
    L.scap_fold_bias_workspace.restype = sz
    L.scap_fold_bias.argtypes = [vp, vp, vp, i, i, i, vp, vp, sz, vp]
    L.scap_fold_bias.restype = i
    L.scap_fc_workspace.argtypes = [i, i, i]
    L.scap_fc_workspace.restype = sz
    L.scap_sparse_fc.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, vp, vp, sz, vp]
    L.scap_sparse_fc.restype = i
    L.scap_dense_fc.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.scap_dense_fc.restype = i
    L.scap_sparse_fc_q8.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, i, i, i, vp, vp, vp, sz, vp]
    L.scap_sparse_fc_q8.restype = i
    L.scap_dense_fc_q8.argtypes = [vp, i, vp, vp, vp, vp, i, i, i, vp, sz, vp]
    L.scap_dense_fc_q8.restype = i
    L.scap_fold_bias_q8.argtypes = [vp, vp, vp, vp, i, i, vp, vp, sz, vp]
    L.scap_fold_bias_q8.restype = i
    L.scap_sparse_fc_q4.argtypes = [vp, i, vp, vp, vp, i, vp, vp, vp, vp, i, i, i, vp, vp, vp, sz, vp]
    L.scap_sparse_fc_q4.restype = i
    L.scap_dense_fc_q4.argtypes = [vp, i, vp, vp, vp, i, vp, vp, i, i, i, vp, sz, vp]
    L.scap_dense_fc_q4.restype = i
    L.scap_fold_bias_q4.argtypes = [vp, vp, vp, i, vp, vp, i, i, vp, vp, sz, vp]
    L.scap_fold_bias_q4.restype = i
    L.scap_grouped_workspace.argtypes = []
    L.scap_grouped_workspace.restype = sz
    L.scap_sparse_fc_grouped.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, C.POINTER(C.c_int), vp, sz, vp]
    L.scap_sparse_fc_grouped.restype = i
    L.scap_fc_host_workspace.argtypes = [i, i, i]
    L.scap_fc_host_workspace.restype = sz
    L.scap_sparse_fc_host.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
    L.scap_sparse_fc_host.restype = i
    L.scap_glu_workspace.argtypes = [i, i, i]
    L.scap_glu_workspace.restype = sz
    L.scap_glu_ffn.argtypes = [vp] * 10 + [i, i, i, i] + [vp] * 5 + [vp, sz, vp]
    L.scap_glu_ffn.restype = i
    L.scap_gelu_ffn_workspace.argtypes = [i, i, i]
    L.scap_gelu_ffn_workspace.restype = sz
    L.scap_gelu_ffn.argtypes = [vp] * 10 + [i, i, i, i] + [vp] * 5 + [vp, sz, vp]
    L.scap_gelu_ffn.restype = i
    L.scap_glu_static_capacity.argtypes = []
    L.scap_glu_static_capacity.restype = sz
    L.scap_glu_ffn_static.argtypes = [vp] * 10 + [i, i, i, i] + [vp, vp]
    L.scap_glu_ffn_static.restype = i
    L.scap_moe_workspace.argtypes = [i, i, i, i, i]
    L.scap_moe_workspace.restype = sz
    L.scap_moe_ffn.argtypes = [vp, vp, C.POINTER(ScapExpert), i, i, vp, i, i, i, i, vp, vp, vp, sz, vp]
    L.scap_moe_ffn.restype = i
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().scap_status_string(int(code)).decode()


def scap_version() -> int:
    return lib().scap_version()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise ScapError(code, where)


def scap_tune(key: str, value: int) -> None:
    _check(lib().scap_tune(key.encode(), int(value)), "scap_tune")


def scap_device_status() -> None:
    """Synchronises the device; raises ScapError(SCAP_ERR_TIMEOUT) if a bounded wait of the tcgen05 kernel ran out."""
    _check(lib().scap_device_status(), "scap_device_status")


def _ptr(t):
    """Address of a tensor's storage, an int address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return SCAP_F16
    if t.dtype == torch.bfloat16:
        return SCAP_BF16
    raise TypeError("weights/activations must be float16 or bfloat16, got %s" % t.dtype)


def _ws(ws):
    return (_ptr(ws), ws.numel() * ws.element_size()) if ws is not None else (None, 0)


def scap_calibrate_workspace(T: int, K: int, nbins: int) -> int:
    return lib().scap_calibrate_workspace(T, K, nbins)


def scap_calibrate(x_calib, sparsity: float, nbins: int, m_out, tau_out, ws, stream=None) -> None:
    T, K = x_calib.shape
    p, n = _ws(ws)
    _check(lib().scap_calibrate(_ptr(x_calib), T, K, dtype_of(x_calib), float(sparsity), nbins, _ptr(m_out), _ptr(tau_out),
                                p, n, _stream(stream)), "scap_calibrate")


SCAP_MODE_HISTOGRAM, SCAP_MODE_MEAN, SCAP_MODE_MEDIAN, SCAP_MODE_KDE = 0, 1, 2, 3
SCAP_ETA_PER_CHANNEL, SCAP_ETA_SCALAR = 0, 1


def scap_calibrate_ex(x_calib, sparsity: float, estimator: int, scope: int, nbins: int, m_out, tau_out, ws, stream=None) -> None:
    T, K = x_calib.shape
    p, n = _ws(ws)
    _check(lib().scap_calibrate_ex(_ptr(x_calib), T, K, dtype_of(x_calib), float(sparsity), int(estimator), int(scope), nbins,
                                   _ptr(m_out), _ptr(tau_out), p, n, _stream(stream)), "scap_calibrate_ex")


def scap_fold_bias_workspace(K: int, N: int) -> int:
    return lib().scap_fold_bias_workspace(K, N)


def scap_fold_bias(W, m, b, b_fused, ws, stream=None) -> None:
    K, N = W.shape
    p, n = _ws(ws)
    _check(lib().scap_fold_bias(_ptr(W), _ptr(m), _ptr(b), K, N, dtype_of(W), _ptr(b_fused), p, n, _stream(stream)),
           "scap_fold_bias")


def scap_fc_workspace(B: int, K: int, N: int) -> int:
    return lib().scap_fc_workspace(B, K, N)


def scap_sparse_fc(x, W, m, tau, b_fused, y, ws, idx_out=None, nnz_out=None, stream=None) -> None:
    B, K = x.shape
    N = W.shape[1]
    p, n = _ws(ws)
    _check(lib().scap_sparse_fc(_ptr(x), _ptr(W), _ptr(m), _ptr(tau), _ptr(b_fused), _ptr(y), B, K, N, dtype_of(W),
                                _ptr(idx_out), _ptr(nnz_out), p, n, _stream(stream)), "scap_sparse_fc")


def scap_dense_fc(x, W, b, y, ws, stream=None) -> None:
    B, K = x.shape
    N = W.shape[1]
    p, n = _ws(ws)
    _check(lib().scap_dense_fc(_ptr(x), _ptr(W), _ptr(b), _ptr(y), B, K, N, dtype_of(W), p, n, _stream(stream)),
           "scap_dense_fc")


def scap_sparse_fc_q8(x, Wq, wscale, m, tau, b_fused, y, ws, idx_out=None, nnz_out=None, stream=None) -> None:
    """Sparse FC on 8-bit weights: Wq int8 [K, N], wscale fp32 [K] (one scale per input channel)."""
    B, K = x.shape
    N = Wq.shape[1]
    p, n = _ws(ws)
    _check(lib().scap_sparse_fc_q8(_ptr(x), dtype_of(x), _ptr(Wq), _ptr(wscale), _ptr(m), _ptr(tau), _ptr(b_fused), _ptr(y), B, K, N,
                                   _ptr(idx_out), _ptr(nnz_out), p, n, _stream(stream)), "scap_sparse_fc_q8")


def scap_dense_fc_q8(x, Wq, wscale, b, y, ws, stream=None) -> None:
    B, K = x.shape
    N = Wq.shape[1]
    p, n = _ws(ws)
    _check(lib().scap_dense_fc_q8(_ptr(x), dtype_of(x), _ptr(Wq), _ptr(wscale), _ptr(b), _ptr(y), B, K, N, p, n, _stream(stream)),
           "scap_dense_fc_q8")


def scap_fold_bias_q8(Wq, wscale, m, b, b_fused, ws, stream=None) -> None:
    K, N = Wq.shape
    p, n = _ws(ws)
    _check(lib().scap_fold_bias_q8(_ptr(Wq), _ptr(wscale), _ptr(m), _ptr(b), K, N, _ptr(b_fused), p, n, _stream(stream)),
           "scap_fold_bias_q8")


def scap_sparse_fc_q4(x, Wq, scale, zero, group, m, tau, b_fused, y, ws, idx_out=None, nnz_out=None, stream=None) -> None:
    """Sparse FC on group-wise 4-bit weights: Wq uint8 [K, N/2] (two codes per byte), scale fp32 and zero uint8 [K/group, N]."""
    B, K = x.shape
    N = Wq.shape[1] * 2
    p, n = _ws(ws)
    _check(lib().scap_sparse_fc_q4(_ptr(x), dtype_of(x), _ptr(Wq), _ptr(scale), _ptr(zero), int(group), _ptr(m), _ptr(tau), _ptr(b_fused),
                                   _ptr(y), B, K, N, _ptr(idx_out), _ptr(nnz_out), p, n, _stream(stream)), "scap_sparse_fc_q4")


def scap_dense_fc_q4(x, Wq, scale, zero, group, b, y, ws, stream=None) -> None:
    B, K = x.shape
    N = Wq.shape[1] * 2
    p, n = _ws(ws)
    _check(lib().scap_dense_fc_q4(_ptr(x), dtype_of(x), _ptr(Wq), _ptr(scale), _ptr(zero), int(group), _ptr(b), _ptr(y), B, K, N, p, n,
                                  _stream(stream)), "scap_dense_fc_q4")


def scap_fold_bias_q4(Wq, scale, zero, group, m, b, b_fused, ws, stream=None) -> None:
    K, N = Wq.shape[0], Wq.shape[1] * 2
    p, n = _ws(ws)
    _check(lib().scap_fold_bias_q4(_ptr(Wq), _ptr(scale), _ptr(zero), int(group), _ptr(m), _ptr(b), K, N, _ptr(b_fused), p, n,
                                   _stream(stream)), "scap_fold_bias_q4")


def scap_grouped_workspace() -> int:
    return lib().scap_grouped_workspace()


def scap_sparse_fc_grouped(x, W, m, tau, b_fused, y, groups, ws, stream=None) -> None:
    """Sparse FC with one union mask per group of rows; ``groups`` is a host sequence of B group numbers 0..15."""
    B, K = x.shape
    N = W.shape[1]
    p, n = _ws(ws)
    arr = (C.c_int * B)(*[int(g) for g in groups])
    _check(lib().scap_sparse_fc_grouped(_ptr(x), _ptr(W), _ptr(m), _ptr(tau), _ptr(b_fused), _ptr(y), B, K, N, dtype_of(W), arr, p, n,
                                        _stream(stream)), "scap_sparse_fc_grouped")


def scap_fc_host_workspace(B: int, K: int, N: int) -> int:
    return lib().scap_fc_host_workspace(B, K, N)


def scap_sparse_fc_host(x_host, W, m, tau, b_fused, y_host, ws, stream=None) -> None:
    """x_host / y_host are CPU tensors (pinned recommended); everything else lives on the device."""
    B, K = x_host.shape
    N = W.shape[1]
    p, n = _ws(ws)
    _check(lib().scap_sparse_fc_host(_ptr(x_host), _ptr(W), _ptr(m), _ptr(tau), _ptr(b_fused), _ptr(y_host), B, K, N,
                                     dtype_of(W), p, n, _stream(stream)), "scap_sparse_fc_host")


def scap_glu_workspace(B: int, D: int, F: int) -> int:
    return lib().scap_glu_workspace(B, D, F)


def scap_glu_ffn(h, Wgu, Wd, m1, tau1, bgu_fused, m2, tau2, bd_fused, y, ws, z_out=None, idx1_out=None, nnz1_out=None,
                 idx2_out=None, nnz2_out=None, stream=None) -> None:
    B, D = h.shape
    F = Wd.shape[0]
    p, n = _ws(ws)
    _check(lib().scap_glu_ffn(_ptr(h), _ptr(Wgu), _ptr(Wd), _ptr(m1), _ptr(tau1), _ptr(bgu_fused), _ptr(m2), _ptr(tau2),
                              _ptr(bd_fused), _ptr(y), B, D, F, dtype_of(Wgu), _ptr(z_out), _ptr(idx1_out), _ptr(nnz1_out),
                              _ptr(idx2_out), _ptr(nnz2_out), p, n, _stream(stream)), "scap_glu_ffn")


def scap_gelu_ffn_workspace(B: int, D: int, F: int) -> int:
    return lib().scap_gelu_ffn_workspace(B, D, F)


def scap_gelu_ffn(h, Wu, Wd, m1, tau1, bu_fused, m2, tau2, bd_fused, y, ws, z_out=None, idx1_out=None, nnz1_out=None,
                  idx2_out=None, nnz2_out=None, stream=None) -> None:
    B, D = h.shape
    F = Wd.shape[0]
    p, n = _ws(ws)
    _check(lib().scap_gelu_ffn(_ptr(h), _ptr(Wu), _ptr(Wd), _ptr(m1), _ptr(tau1), _ptr(bu_fused), _ptr(m2), _ptr(tau2),
                               _ptr(bd_fused), _ptr(y), B, D, F, dtype_of(Wu), _ptr(z_out), _ptr(idx1_out), _ptr(nnz1_out),
                               _ptr(idx2_out), _ptr(nnz2_out), p, n, _stream(stream)), "scap_gelu_ffn")


def scap_glu_static_capacity() -> int:
    return lib().scap_glu_static_capacity()


def scap_glu_ffn_static(h, Wgu, Wd, m1, tau1, bgu_fused, m2, tau2, bd_fused, y, z_out=None, stream=None) -> None:
    """scap_glu_ffn for callers that may not allocate: the scratch is a fixed array inside the library (see scap.h)."""
    B, D = h.shape
    F = Wd.shape[0]
    _check(lib().scap_glu_ffn_static(_ptr(h), _ptr(Wgu), _ptr(Wd), _ptr(m1), _ptr(tau1), _ptr(bgu_fused), _ptr(m2),
                                     _ptr(tau2), _ptr(bd_fused), _ptr(y), B, D, F, dtype_of(Wgu), _ptr(z_out),
                                     _stream(stream)), "scap_glu_ffn_static")


def scap_moe_workspace(B: int, D: int, F: int, E: int, top_k: int) -> int:
    return lib().scap_moe_workspace(B, D, F, E, top_k)


def scap_moe_ffn(h, logits, experts, top_k: int, y, ws, expert_out=None, weight_out=None, stream=None) -> None:
    """``experts``: list of dicts of tensors with the fields of ``scap_expert`` (None where nullable)."""
    B, D = h.shape
    E = len(experts)
    F = experts[0]["Wd"].shape[0]
    arr = (ScapExpert * E)()
    for e, p_ in enumerate(experts):
        for name, _ in ScapExpert._fields_:
            setattr(arr[e], name, _ptr(p_.get(name)))
    p, n = _ws(ws)
    _check(lib().scap_moe_ffn(_ptr(h), _ptr(logits), arr, E, top_k, _ptr(y), B, D, F, dtype_of(h), _ptr(expert_out),
                              _ptr(weight_out), p, n, _stream(stream)), "scap_moe_ffn")
