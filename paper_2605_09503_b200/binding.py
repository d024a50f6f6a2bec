"""Thin Python binding of the C ABI declared in include/pq.h.

Argument marshalling only: every function takes torch CUDA tensors (used for device memory
and the current stream, nothing else), checks dtypes, and forwards raw pointers and sizes to
the entry point of the same name in libpq.so.  There is no fallback: if the library is
missing or the call fails, an exception is raised.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpq.so")

PQ_OK = 0
PQ_SF_LINEAR, PQ_SF_TCGEN05 = 0, 1
OP_CALIB_STATS, OP_SELECT_PERM, OP_GROUP_ERROR, OP_QUANT_WEIGHT, OP_GEMM, OP_OUTPUT_ERROR = 1, 2, 3, 4, 5, 6
CHUNK_ROWS = 16
KIND_NVFP4, KIND_INT = 0, 1


class PqError(RuntimeError):
    def __init__(self, name, code, text):
        super().__init__(f"{name} failed: status {code} ({text})")
        self.code = code


class pq_format(C.Structure):
    _fields_ = [("kind", C.c_int), ("bits", C.c_int), ("group", C.c_int)]


_lib = None
_vp, _i64, _sz, _int = C.c_void_p, C.c_int64, C.c_size_t, C.c_int

_SIGNATURES = {
    "pq_status_string": (C.c_char_p, [_int]),
    "pq_version": (_int, []),
    "pq_workspace_bytes": (_sz, [_int, _i64, _i64, _i64, _int]),
    "pq_sf_bytes": (_sz, [_i64, _i64, _int]),
    "pq_calib_stats": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _sz, _vp]),
    "pq_quant_act_nvfp4_perm": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _int, _vp]),
    "pq_order_by_absmax": (_int, [_vp, _i64, _vp, _vp, _sz, _vp]),
    "pq_calib_sum": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _sz, _vp]),
    "pq_order_by_variance": (_int, [_vp, _vp, _i64, _i64, _vp, _vp, _sz, _vp]),
    "pq_order_round_robin": (_int, [_vp, _i64, _int, _vp, _vp, _sz, _vp]),
    "pq_output_error": (_int, [_vp, _i64, _vp, _i64, _i64, _i64, _vp, _vp, _sz, _vp]),
    "pq_calib_stats_static": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "pq_calib_stats_static_max_bytes": (_sz, []),
    "pq_tensor_scale": (_int, [_vp, _i64, _vp, _vp]),
    "pq_select_perm": (_int, [_vp, _i64, _vp, _i64, _i64, _int, _vp, _vp, _sz, _vp]),
    "pq_group_error": (_int, [_vp, _i64, _i64, _i64, pq_format, _vp, _vp, _int, _vp, _vp, _sz, _vp]),
    "pq_error_weights": (_int, [_vp, _vp, _i64, _vp, _vp]),
    "pq_accept": (_int, [_vp, _vp, _vp, _int, _i64, C.c_double, _vp, _vp, _vp, _vp]),
    "pq_quant_weight": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _int, _vp, _vp, _sz, _vp]),
    "pq_quant_act_nvfp4": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _int, _vp]),
    "pq_gemm_w4a4": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _i64, _vp, _sz, _vp]),
    "pq_linear_w4a4": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64,
                              _vp, _sz, _vp]),
    "pq_linear_w4a4_batched": (_int, [_int, _vp, _i64, _i64, _i64, _vp, _vp, _vp, _int, _vp, _vp, _vp, _i64, _vp, _i64,
                                      _vp, _sz, _vp]),
    "pq_linear_w4a4_host_batched": (_int, [_int, _vp, _i64, _i64, _vp, _vp, _vp, _int, _vp, _vp, _vp, _vp, _vp, _i64, _vp,
                                           _vp, _sz, _vp]),
    "pq_linear_w4a4_host": (_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _vp,
                                   _vp, _sz, _vp]),
    "pq_fakequant_int": (_int, [_vp, _i64, _i64, _i64, pq_format, _vp, _vp, _i64, _vp]),
    "pq_sf_to_linear": (_int, [_vp, _i64, _i64, _vp, _vp]),
    "pq_norm_quant_nvfp4": (_int, [_vp, _i64, _i64, _i64, _int, _vp, _vp, C.c_float, _vp, _vp, _vp, _vp, _int, _vp,
                                   _vp]),
    "pq_hadamard_quant_nvfp4": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _int, _vp, _vp]),
    "pq_last_error_detail": (C.c_char_p, []),
    "pq_device_status": (_int, [_vp, _vp]),
    "pq_selftest_wait_expiry": (_int, [_vp, _sz, C.c_longlong, _vp, _vp]),
}


def lib():
    """Load libpq.so (built in-tree by paper_2605_09503_b200/build.py).  Fails loudly."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: run `python -m paper_2605_09503_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            if not hasattr(L, name):
                continue  # reported by the symbol test; calling it raises AttributeError
            f = getattr(L, name)
            f.restype, f.argtypes = res, args
        _lib = L
    return _lib


def status_string(code):
    return lib().pq_status_string(code).decode()


def _check(name, code):
    if code != PQ_OK:
        detail = status_string(code)
        if code == 6:   # PQ_ERR_CUDA: say which call failed
            extra = lib().pq_last_error_detail()
            if extra:
                detail += " -- " + extra.decode()
        raise PqError(name, code, detail)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _p(t):
    if t is None:
        return None
    assert t.is_cuda, "device tensors only"
    return C.c_void_p(t.data_ptr())


def _bf16(t):
    assert t.dtype == torch.bfloat16 and t.dim() == 2 and t.stride(1) == 1
    return t


def workspace_bytes(op, rows, K, N=0, P=0):
    return int(lib().pq_workspace_bytes(op, rows, K, N, P))


def sf_bytes(rows, K, layout):
    return int(lib().pq_sf_bytes(rows, K, layout))


def workspace(op, rows, K, N=0, P=0, device="cuda"):
    """Allocate (through torch) a workspace big enough for the given call."""
    return torch.zeros(max(workspace_bytes(op, rows, K, N, P), 256), dtype=torch.uint8, device=device)


def _ws(ws):
    return _p(ws), (ws.numel() if ws is not None else 0)


# ---------------------------------------------------------------------------- entry points
def pq_calib_stats(T, sumsq, amax, ws):
    _bf16(T)
    assert sumsq.dtype == torch.float64 and amax.dtype == torch.float32
    w, wb = _ws(ws)
    _check("pq_calib_stats", lib().pq_calib_stats(_p(T), T.shape[0], T.shape[1], T.stride(0), _p(sumsq),
                                                  _p(amax), w, wb, _stream()))


def pq_order_by_absmax(amax, perm, ws):
    """perm[pos] = channel with the pos-th largest absmax (ties by ascending channel); int32 [K]."""
    assert amax.dtype == torch.float32 and perm.dtype == torch.int32 and perm.numel() == amax.numel()
    w, wb = _ws(ws)
    _check("pq_order_by_absmax", lib().pq_order_by_absmax(_p(amax), amax.numel(), _p(perm), w, wb, _stream()))


def pq_calib_sum(T, total, ws):
    """total[i] += sum over rows of T[:, i] (fp64 [K]); workspace as for pq_calib_stats."""
    _bf16(T)
    assert total.dtype == torch.float64 and total.numel() == T.shape[1]
    w, wb = _ws(ws)
    _check("pq_calib_sum", lib().pq_calib_sum(_p(T), T.shape[0], T.shape[1], T.stride(0), _p(total), w, wb, _stream()))


def pq_order_by_variance(total, sumsq, rows, perm, ws):
    """perm[pos] = channel with the pos-th largest variance sumsq/rows - (total/rows)^2; int32 [K]."""
    assert total.dtype == torch.float64 and sumsq.dtype == torch.float64 and perm.dtype == torch.int32
    assert total.numel() == sumsq.numel() == perm.numel()
    w, wb = _ws(ws)
    _check("pq_order_by_variance", lib().pq_order_by_variance(_p(total), _p(sumsq), int(rows), sumsq.numel(), _p(perm),
                                                              w, wb, _stream()))


def pq_order_round_robin(sumsq, group, perm, ws):
    """Channels sorted by descending second moment, dealt to the K / group groups in turn; int32 [K]."""
    assert sumsq.dtype == torch.float64 and perm.dtype == torch.int32 and perm.numel() == sumsq.numel()
    w, wb = _ws(ws)
    _check("pq_order_round_robin", lib().pq_order_round_robin(_p(sumsq), sumsq.numel(), int(group), _p(perm), w, wb,
                                                              _stream()))


def pq_output_error(Yref, Yq, err, ws):
    """err[n] += sum over rows of (Yref - Yq)^2: Yref fp32 [rows, N], Yq bf16 [rows, N], err fp64 [N]."""
    _bf16(Yq)
    assert Yref.dtype == torch.float32 and Yref.dim() == 2 and Yref.stride(1) == 1 and Yref.shape == Yq.shape
    assert err.dtype == torch.float64 and err.numel() == Yq.shape[1]
    w, wb = _ws(ws)
    _check("pq_output_error", lib().pq_output_error(_p(Yref), Yref.stride(0), _p(Yq), Yq.stride(0), Yq.shape[0],
                                                    Yq.shape[1], _p(err), w, wb, _stream()))


def pq_calib_stats_static(T, sumsq, amax):
    """pq_calib_stats without a workspace argument: for callers that may not allocate device
    memory, the partial sums live in a fixed 8 MiB array inside the library (one per GPU).  Raises
    PqError (workspace) when the problem needs more than that; calls that overlap on the GPU race."""
    _bf16(T)
    assert sumsq.dtype == torch.float64 and amax.dtype == torch.float32
    _check("pq_calib_stats_static", lib().pq_calib_stats_static(_p(T), T.shape[0], T.shape[1], T.stride(0),
                                                                _p(sumsq), _p(amax), _stream()))


def pq_tensor_scale(amax, ts):
    assert amax.dtype == torch.float32 and ts.dtype == torch.float32
    _check("pq_tensor_scale", lib().pq_tensor_scale(_p(amax), amax.numel(), _p(ts), _stream()))


def pq_select_perm(sumsq_a, rows_a, sumsq_w, rows_w, J, perms, ws):
    assert sumsq_a.dtype == torch.float64 and sumsq_w.dtype == torch.float64 and perms.dtype == torch.int32
    K = sumsq_a.numel()
    assert perms.shape == (J + 1, K) and perms.is_contiguous()
    w, wb = _ws(ws)
    _check("pq_select_perm", lib().pq_select_perm(_p(sumsq_a), rows_a, _p(sumsq_w), rows_w, K, J, _p(perms),
                                                  w, wb, _stream()))


def pq_group_error(T, fmt, ts, perms, err, ws):
    _bf16(T)
    kind, bits, group = fmt
    P = 1 if perms is None else perms.shape[0]
    if perms is not None:
        assert perms.dtype == torch.int32 and perms.is_contiguous() and perms.shape[1] == T.shape[1]
    assert err.dtype == torch.float64 and err.is_contiguous()
    w, wb = _ws(ws)
    _check("pq_group_error", lib().pq_group_error(_p(T), T.shape[0], T.shape[1], T.stride(0),
                                                  pq_format(kind, bits, group), _p(ts), _p(perms), P, _p(err),
                                                  w, wb, _stream()))


def pq_error_weights(sumsq_a, sumsq_w, lam):
    assert lam.dtype == torch.float64 and lam.numel() == 2
    _check("pq_error_weights", lib().pq_error_weights(_p(sumsq_a), _p(sumsq_w), sumsq_a.numel(), _p(lam),
                                                      _stream()))


def pq_accept(err_x, err_w, lam, tau, best, accept, E=None):
    assert err_x.dtype == torch.float64 and err_w.dtype == torch.float64 and err_x.shape == err_w.shape
    assert err_x.is_contiguous() and err_w.is_contiguous()
    assert best.dtype == torch.int32 and accept.dtype == torch.int32
    P, Kg = err_x.shape[0] - 1, err_x.shape[1]
    _check("pq_accept", lib().pq_accept(_p(err_x), _p(err_w), _p(lam), P, Kg, float(tau), _p(best), _p(accept),
                                        _p(E), _stream()))


def pq_quant_weight(Wt, perm, perm_select, codes, sf, sf_layout, ts_w, ws):
    _bf16(Wt)
    assert codes.dtype == torch.uint8 and sf.dtype == torch.uint8 and ts_w.dtype == torch.float32
    w, wb = _ws(ws)
    _check("pq_quant_weight", lib().pq_quant_weight(_p(Wt), Wt.shape[0], Wt.shape[1], Wt.stride(0), _p(perm),
                                                    _p(perm_select), _p(codes), _p(sf), sf_layout, _p(ts_w),
                                                    w, wb, _stream()))


def pq_quant_act_nvfp4(X, ts_x, codes, sf, sf_layout):
    _bf16(X)
    assert codes.dtype == torch.uint8 and sf.dtype == torch.uint8 and ts_x.dtype == torch.float32
    _check("pq_quant_act_nvfp4", lib().pq_quant_act_nvfp4(_p(X), X.shape[0], X.shape[1], X.stride(0), _p(ts_x),
                                                          _p(codes), _p(sf), sf_layout, _stream()))


def pq_quant_act_nvfp4_perm(X, perm, ts_x, codes, sf, sf_layout):
    """Codes and scales of X with its channels taken in the order `perm` (int32 [K], or None)."""
    _bf16(X)
    assert codes.dtype == torch.uint8 and sf.dtype == torch.uint8 and ts_x.dtype == torch.float32
    assert perm is None or (perm.dtype == torch.int32 and perm.numel() == X.shape[1] and perm.is_contiguous())
    _check("pq_quant_act_nvfp4_perm", lib().pq_quant_act_nvfp4_perm(_p(X), X.shape[0], X.shape[1], X.stride(0),
                                                                    _p(perm), _p(ts_x), _p(codes), _p(sf),
                                                                    sf_layout, _stream()))


def pq_gemm_w4a4(xq, sfx, ts_x, wq, sfw, ts_w, Y, ws):
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    assert Y.dtype == torch.bfloat16 and Y.shape == (M, N) and Y.stride(1) == 1
    w, wb = _ws(ws)
    _check("pq_gemm_w4a4", lib().pq_gemm_w4a4(_p(xq), _p(sfx), _p(ts_x), _p(wq), _p(sfw), _p(ts_w), M, N, K,
                                              _p(Y), Y.stride(0), w, wb, _stream()))


def pq_linear_w4a4(X, ts_x, xq, sfx, wq, sfw, ts_w, Y, ws):
    _bf16(X)
    M, K = X.shape
    N = wq.shape[0]
    assert Y.dtype == torch.bfloat16 and Y.shape == (M, N) and Y.stride(1) == 1
    w, wb = _ws(ws)
    _check("pq_linear_w4a4", lib().pq_linear_w4a4(_p(X), M, K, X.stride(0), _p(ts_x), _p(xq), _p(sfx), _p(wq),
                                                  _p(sfw), _p(ts_w), N, _p(Y), Y.stride(0), w, wb, _stream()))


def pq_linear_w4a4_batched(Xs, ts_x, xqs, sfxs, wq, sfw, ts_w, Ys, ws):
    """n batches through one layer; Xs / Ys lists of n tensors, xqs / sfxs lists of n_sets intermediates."""
    n, n_sets = len(Xs), len(xqs)
    assert len(Ys) == n and len(sfxs) == n_sets
    M, K = Xs[0].shape
    N = wq.shape[0]
    for x, y in zip(Xs, Ys):
        _bf16(x)
        assert x.shape == (M, K) and x.stride(0) == Xs[0].stride(0)
        assert y.dtype == torch.bfloat16 and y.shape == (M, N) and y.stride(1) == 1 and y.stride(0) == Ys[0].stride(0)
    arr = lambda ts: (C.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
    w, wb = _ws(ws)
    _check("pq_linear_w4a4_batched", lib().pq_linear_w4a4_batched(
        n, arr(Xs), M, K, Xs[0].stride(0), _p(ts_x), arr(xqs), arr(sfxs), n_sets, _p(wq), _p(sfw), _p(ts_w), N,
        arr(Ys), Ys[0].stride(0), w, wb, _stream()))


def pq_linear_w4a4_host_batched(X_hosts, ts_x, X_devs, Y_devs, xq, sfx, wq, sfw, ts_w, Y_hosts, ws):
    """n host batches in, n host batches out; uploads, kernels and downloads of neighbouring batches overlap."""
    n, n_sets = len(X_hosts), len(X_devs)
    assert len(Y_hosts) == n and len(Y_devs) == n_sets
    M, K = X_hosts[0].shape
    N = wq.shape[0]
    for x, y in zip(X_hosts, Y_hosts):
        assert not x.is_cuda and not y.is_cuda and x.is_contiguous() and y.is_contiguous()
        assert x.dtype == torch.bfloat16 and y.dtype == torch.bfloat16 and x.shape == (M, K) and y.shape == (M, N)
    for x, y in zip(X_devs, Y_devs):
        _bf16(x)
        assert x.shape == (M, K) and x.is_contiguous() and y.shape == (M, N) and y.is_contiguous() and y.is_cuda
    arr = lambda ts: (C.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
    w, wb = _ws(ws)
    _check("pq_linear_w4a4_host_batched", lib().pq_linear_w4a4_host_batched(
        n, arr(X_hosts), M, K, _p(ts_x), arr(X_devs), arr(Y_devs), n_sets, _p(xq), _p(sfx), _p(wq), _p(sfw), _p(ts_w),
        N, arr(Y_hosts), w, wb, _stream()))


def pq_linear_w4a4_host(X_host, ts_x, X_dev, xq, sfx, wq, sfw, ts_w, Y_dev, Y_host, ws):
    """Host tensors in, host tensor out (pinned CPU tensors); copies and kernels are enqueued on
    the current stream, the caller synchronises before reading Y_host."""
    assert not X_host.is_cuda and not Y_host.is_cuda and X_host.is_contiguous() and Y_host.is_contiguous()
    assert X_host.dtype == torch.bfloat16 and Y_host.dtype == torch.bfloat16
    _bf16(X_dev)
    M, K = X_host.shape
    N = wq.shape[0]
    assert X_dev.shape == (M, K) and X_dev.is_contiguous() and Y_dev.shape == (M, N) and Y_dev.is_contiguous()
    assert Y_host.shape == (M, N)
    w, wb = _ws(ws)
    _check("pq_linear_w4a4_host", lib().pq_linear_w4a4_host(
        C.c_void_p(X_host.data_ptr()), M, K, _p(ts_x), _p(X_dev), _p(xq), _p(sfx), _p(wq), _p(sfw), _p(ts_w), N,
        _p(Y_dev), C.c_void_p(Y_host.data_ptr()), w, wb, _stream()))


def pq_fakequant_int(T, fmt, perm, out):
    _bf16(T)
    _bf16(out)
    kind, bits, group = fmt
    _check("pq_fakequant_int", lib().pq_fakequant_int(_p(T), T.shape[0], T.shape[1], T.stride(0),
                                                      pq_format(kind, bits, group), _p(perm), _p(out),
                                                      out.stride(0), _stream()))


def pq_sf_to_linear(sf_tc, rows, K, sf_linear):
    _check("pq_sf_to_linear", lib().pq_sf_to_linear(_p(sf_tc), rows, K, _p(sf_linear), _stream()))


NORM_RMS, NORM_ADALN = 0, 1


def pq_norm_quant_nvfp4(H, kind, a, b, eps, perm, ts_x, codes, sf, sf_layout, y_out=None):
    _bf16(H)
    M, K = H.shape
    assert a.dtype == torch.float32 and a.numel() == K and (b is None or (b.dtype == torch.float32 and b.numel() == K))
    assert perm is None or (perm.dtype == torch.int32 and perm.numel() == K)
    assert y_out is None or (y_out.dtype == torch.bfloat16 and y_out.shape == (M, K) and y_out.is_contiguous())
    _check("pq_norm_quant_nvfp4", lib().pq_norm_quant_nvfp4(_p(H), M, K, H.stride(0), kind, _p(a), _p(b), eps, _p(perm),
                                                            _p(ts_x), _p(codes), _p(sf), sf_layout, _p(y_out), _stream()))


def pq_hadamard_quant_nvfp4(X, perm, ts_x, codes, sf, sf_layout, y_out=None):
    """Rows of X through the Hadamard transform, channels read in the order perm, NVFP4 codes and scales of
    the result (codes = sf = None: transform only, into y_out)."""
    _bf16(X)
    M, K = X.shape
    assert perm is None or (perm.dtype == torch.int32 and perm.numel() == K and perm.is_contiguous())
    assert (codes is None) == (sf is None)
    assert codes is None or (codes.dtype == torch.uint8 and sf.dtype == torch.uint8 and ts_x.dtype == torch.float32)
    assert y_out is None or (y_out.dtype == torch.bfloat16 and y_out.shape == (M, K) and y_out.is_contiguous())
    _check("pq_hadamard_quant_nvfp4", lib().pq_hadamard_quant_nvfp4(_p(X), M, K, X.stride(0), _p(perm), _p(ts_x),
                                                                    _p(codes), _p(sf), sf_layout, _p(y_out), _stream()))


def pq_device_status(ws):
    return int(lib().pq_device_status(_p(ws), _stream()))


def pq_selftest_wait_expiry(ws, limit_cycles):
    """A bounded device-side wait that is left to run out; -> (wait result, abort flag) as the kernel saw them."""
    observed = torch.full((2,), -1, dtype=torch.int32, device=ws.device)
    w, wb = _ws(ws)
    _check("pq_selftest_wait_expiry", lib().pq_selftest_wait_expiry(w, wb, int(limit_cycles), _p(observed), _stream()))
    return tuple(observed.tolist())
