"""numpy front-end of the C oracle (oracle/pq_oracle.c).  Test infrastructure only.

bf16 tensors travel as uint16 numpy arrays (raw bit patterns); everything else is plain numpy.
Each function mirrors one C routine and cites the same passage of the paper as that routine.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _declare(_lib)
    return _lib


_P = C.c_void_p
_i64 = C.c_int64


def _declare(L):
    L.pqo_bf16_to_f32.restype = C.c_float
    L.pqo_bf16_to_f32.argtypes = [C.c_uint16]
    L.pqo_f32_to_bf16.restype = C.c_uint16
    L.pqo_f32_to_bf16.argtypes = [C.c_float]
    L.pqo_e2m1_value.restype = C.c_float
    L.pqo_e2m1_value.argtypes = [C.c_uint8]
    L.pqo_e2m1_encode_abs.restype = C.c_uint8
    L.pqo_e2m1_encode_abs.argtypes = [C.c_float]
    L.pqo_e4m3_value.restype = C.c_float
    L.pqo_e4m3_value.argtypes = [C.c_uint8]
    L.pqo_e4m3_encode.restype = C.c_uint8
    L.pqo_e4m3_encode.argtypes = [C.c_float]
    L.pqo_tensor_scale.restype = C.c_float
    L.pqo_tensor_scale.argtypes = [_P, _i64]
    L.pqo_calib_stats.argtypes = [_P, _i64, _i64, _i64, _P, _P]
    L.pqo_select_perm.argtypes = [_P, _i64, _P, _i64, _i64, C.c_int, _P]
    L.pqo_output_error.argtypes = [_P, _i64, _P, _i64, _i64, _i64, _P]
    L.pqo_order_by_absmax.argtypes = [_P, _i64, _P]
    L.pqo_calib_sum.argtypes = [_P, _i64, _i64, _i64, _P]
    L.pqo_order_by_variance.argtypes = [_P, _P, _i64, _i64, _P]
    L.pqo_order_round_robin.argtypes = [_P, _i64, C.c_int, _P]
    L.pqo_group_error.argtypes = [_P, _i64, _i64, _i64, C.c_int, C.c_int, C.c_int, C.c_float, _P,
                                  C.c_int, _P]
    L.pqo_accept.argtypes = [_P, C.c_double, _P, C.c_double, C.c_int, _i64, C.c_double, _P, _P, _P]
    L.pqo_error_weight.restype = C.c_double
    L.pqo_error_weight.argtypes = [_P, _i64]
    L.pqo_quant_nvfp4.argtypes = [_P, _i64, _i64, _i64, _P, C.c_float, _P, _P]
    L.pqo_dequant_nvfp4.argtypes = [_P, _P, C.c_float, _i64, _i64, _P]
    L.pqo_norm_quant_nvfp4.argtypes = [_P, _i64, _i64, _i64, C.c_int, _P, _P, C.c_float, _P, C.c_float, _P, _P, _P]
    L.pqo_hadamard_quant_nvfp4.argtypes = [_P, _i64, _i64, _i64, _P, C.c_float, _P, _P, _P, _P]
    L.pqo_fakequant_int.argtypes = [_P, _i64, _i64, _i64, C.c_int, C.c_int, _P, _P, _i64]
    L.pqo_gemm_ref_one.restype = C.c_double
    L.pqo_gemm_ref_one.argtypes = [_P, _P, C.c_float, _P, _P, C.c_float, _i64, _i64, _i64]
    L.pqo_gemm_ref.argtypes = [_P, _P, C.c_float, _P, _P, C.c_float, _i64, _i64, _i64, _P]
    L.pqo_gemm_ref_sampled.argtypes = [_P, _P, C.c_float, _P, _P, C.c_float, _i64, _P, _P, _i64, _P]
    L.pqo_gemm_bf16_ref.argtypes = [_P, _P, _i64, _i64, _i64, _P, _P]
    L.pqo_chunk_rows.restype = C.c_int
    L.pqo_slab_rows.restype = C.c_int


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _bf16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16 and a.ndim == 2, "bf16 tensors are passed as 2-D uint16 bit patterns"
    return a


def _perm(p, K, nrows=None):
    if p is None:
        return None
    p = np.ascontiguousarray(p, dtype=np.int32)
    assert p.shape[-1] == K
    return p


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what}: invalid arguments (code {rc})")


# ---------------------------------------------------------------- scalar formats
def bf16_to_f32(bits):
    """Exact widening of bf16 bit patterns (uint16 array) to float32."""
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x):
    """Round-to-nearest-even narrowing, element by element through the C routine."""
    x = np.asarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    L = lib()
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = L.pqo_f32_to_bf16(float(flat_in[i]))
    return out


def e2m1_value(code):
    return float(lib().pqo_e2m1_value(int(code)))


def e2m1_encode_abs(ay):
    return int(lib().pqo_e2m1_encode_abs(float(ay)))


def e4m3_value(code):
    return float(lib().pqo_e4m3_value(int(code)))


def e4m3_encode(u):
    return int(lib().pqo_e4m3_encode(float(u)))


def tensor_scale(amax):
    amax = np.ascontiguousarray(amax, dtype=np.float32)
    return float(lib().pqo_tensor_scale(_ptr(amax), amax.size))


# ---------------------------------------------------------------- pipeline steps
def calib_stats(T, sumsq=None, amax=None):
    """Accumulate per-channel sum of squares (fp64) and absmax (fp32) of one batch."""
    T = _bf16(T)
    rows, K = T.shape
    if sumsq is None:
        sumsq = np.zeros(K, dtype=np.float64)
    if amax is None:
        amax = np.zeros(K, dtype=np.float32)
    _check(lib().pqo_calib_stats(_ptr(T), rows, K, K, _ptr(sumsq), _ptr(amax)), "calib_stats")
    return sumsq, amax


def output_error(Yref, Yq, err=None):
    """Sec. 3.3 / Eq. 10, output-side reading: per output column the sum over rows of
    (Yref - Yq)^2, Yref fp32 [rows, N], Yq bf16 bit patterns [rows, N]; accumulated into err (fp64 [N])."""
    Yref = np.ascontiguousarray(Yref, dtype=np.float32)
    Yq = _bf16(Yq)
    rows, N = Yref.shape
    assert Yq.shape == (rows, N)
    if err is None:
        err = np.zeros(N, dtype=np.float64)
    _check(lib().pqo_output_error(_ptr(Yref), N, _ptr(Yq), N, rows, N, _ptr(err)), "output_error")
    return err


def select_perm(sumsq_a, rows_a, sumsq_w, rows_w, J=5):
    """Eq. 9 candidates for alpha = j/J: int32 [J+1, K], row j sorted by descending key."""
    sumsq_a = np.ascontiguousarray(sumsq_a, dtype=np.float64)
    sumsq_w = np.ascontiguousarray(sumsq_w, dtype=np.float64)
    K = sumsq_a.size
    perms = np.empty((J + 1, K), dtype=np.int32)
    _check(lib().pqo_select_perm(_ptr(sumsq_a), rows_a, _ptr(sumsq_w), rows_w, K, J, _ptr(perms)),
           "select_perm")
    return perms


def order_by_absmax(amax):
    """Tab. 2(a) absmax criterion: channels by descending absmax, ties by ascending channel (int32 [K])."""
    amax = np.ascontiguousarray(amax, dtype=np.float32)
    perm = np.empty(amax.size, dtype=np.int32)
    _check(lib().pqo_order_by_absmax(_ptr(amax), amax.size, _ptr(perm)), "order_by_absmax")
    return perm


def calib_sum(T, total=None):
    """Accumulate the per-channel plain sum (fp64) of one batch: the first moment of the variance criterion."""
    T = _bf16(T)
    rows, K = T.shape
    if total is None:
        total = np.zeros(K, dtype=np.float64)
    _check(lib().pqo_calib_sum(_ptr(T), rows, K, K, _ptr(total)), "calib_sum")
    return total


def order_by_variance(total, sumsq, rows):
    """Tab. 2(a) variance criterion: channels by descending E[x^2] - E[x]^2, ties by ascending channel."""
    total = np.ascontiguousarray(total, dtype=np.float64)
    sumsq = np.ascontiguousarray(sumsq, dtype=np.float64)
    perm = np.empty(sumsq.size, dtype=np.int32)
    _check(lib().pqo_order_by_variance(_ptr(total), _ptr(sumsq), int(rows), sumsq.size, _ptr(perm)), "order_by_variance")
    return perm


def order_round_robin(sumsq, group):
    """Tab. 2(a) round-robin order (this build's reading): channels sorted by descending second moment and
    dealt to the K / group groups in turn."""
    sumsq = np.ascontiguousarray(sumsq, dtype=np.float64)
    perm = np.empty(sumsq.size, dtype=np.int32)
    _check(lib().pqo_order_round_robin(_ptr(sumsq), sumsq.size, int(group), _ptr(perm)), "order_round_robin")
    return perm


def group_error(T, kind, bits, group, ts=1.0, perms=None, err=None):
    """Eq. 3 per candidate and group column, accumulated into err [P, K/group] (fp64)."""
    T = _bf16(T)
    rows, K = T.shape
    if perms is not None:
        perms = _perm(perms, K)
        if perms.ndim == 1:
            perms = perms[None, :]
        P = perms.shape[0]
    else:
        P = 1
    if err is None:
        err = np.zeros((P, K // group), dtype=np.float64)
    assert err.shape == (P, K // group) and err.dtype == np.float64 and err.flags.c_contiguous
    _check(lib().pqo_group_error(_ptr(T), rows, K, K, kind, bits, group, C.c_float(ts), _ptr(perms),
                                 P, _ptr(err)), "group_error")
    return err


def accept(err_x, lambda_x, err_w, lambda_w, tau=0.0):
    """Eq. 10.  err_* are [P+1, Kg] with row 0 the original order.  -> (best, accept, E[P+1])."""
    err_x = np.ascontiguousarray(err_x, dtype=np.float64)
    err_w = np.ascontiguousarray(err_w, dtype=np.float64)
    P = err_x.shape[0] - 1
    Kg = err_x.shape[1]
    assert err_w.shape == err_x.shape
    best = np.zeros(1, dtype=np.int32)
    acc = np.zeros(1, dtype=np.int32)
    E = np.zeros(P + 1, dtype=np.float64)
    _check(lib().pqo_accept(_ptr(err_x), lambda_x, _ptr(err_w), lambda_w, P, Kg, tau, _ptr(best),
                            _ptr(acc), _ptr(E)), "accept")
    return int(best[0]), int(acc[0]), E


def error_weight(sumsq):
    sumsq = np.ascontiguousarray(sumsq, dtype=np.float64)
    return float(lib().pqo_error_weight(_ptr(sumsq), sumsq.size))


def quant_nvfp4(T, ts, perm=None):
    """-> (codes uint8 [rows, K/2], scale bytes uint8 [rows, K/16]) of T[:, perm]."""
    T = _bf16(T)
    rows, K = T.shape
    perm = _perm(perm, K)
    codes = np.empty((rows, K // 2), dtype=np.uint8)
    sf = np.empty((rows, K // 16), dtype=np.uint8)
    _check(lib().pqo_quant_nvfp4(_ptr(T), rows, K, K, _ptr(perm), C.c_float(ts), _ptr(codes),
                                 _ptr(sf)), "quant_nvfp4")
    return codes, sf


def norm_quant_nvfp4(H, kind, a, b, eps, ts, perm=None):
    """Fused normalization (0 = RMSNorm with weight a, 1 = adaptive LayerNorm with scale a, shift b; a and b
    indexed by output position), reordering and NVFP4 quantization
    -> (codes, scale bytes [rows, K/16], bf16 bits of the reordered output)."""
    H = _bf16(H)
    rows, K = H.shape
    perm = _perm(perm, K)
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = None if b is None else np.ascontiguousarray(b, dtype=np.float32)
    codes = np.empty((rows, K // 2), dtype=np.uint8)
    sf = np.empty((rows, K // 16), dtype=np.uint8)
    y = np.empty((rows, K), dtype=np.uint16)
    _check(lib().pqo_norm_quant_nvfp4(_ptr(H), rows, K, K, kind, _ptr(a), _ptr(b), C.c_float(eps), _ptr(perm),
                                      C.c_float(ts), _ptr(codes), _ptr(sf), _ptr(y)), "norm_quant_nvfp4")
    return codes, sf, y


def hadamard_quant_nvfp4(X, ts, perm=None, quantize=True):
    """App. D: rows of X through the Hadamard transform, channels read in the order perm, NVFP4 groups of
    the fp32 result.  -> (codes, sf, y_bf16 bits, y_f32); codes / sf are None with quantize=False."""
    X = _bf16(X)
    rows, K = X.shape
    perm = _perm(perm, K)
    codes = np.empty((rows, K // 2), dtype=np.uint8) if quantize else None
    sf = np.empty((rows, K // 16), dtype=np.uint8) if quantize else None
    y = np.empty((rows, K), dtype=np.uint16)
    yf = np.empty((rows, K), dtype=np.float32)
    _check(lib().pqo_hadamard_quant_nvfp4(_ptr(X), rows, K, K, _ptr(perm), C.c_float(ts), _ptr(codes), _ptr(sf), _ptr(y),
                                          _ptr(yf)), "hadamard_quant_nvfp4")
    return codes, sf, y, yf


def dequant_nvfp4(codes, sf, ts):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    sf = np.ascontiguousarray(sf, dtype=np.uint8)
    rows, K = codes.shape[0], codes.shape[1] * 2
    out = np.empty((rows, K), dtype=np.float32)
    _check(lib().pqo_dequant_nvfp4(_ptr(codes), _ptr(sf), C.c_float(ts), rows, K, _ptr(out)),
           "dequant_nvfp4")
    return out


def fakequant_int(T, bits, group, perm=None):
    """Eq. 1-2 quantize-dequantize of T[:, perm], result as bf16 bit patterns."""
    T = _bf16(T)
    rows, K = T.shape
    perm = _perm(perm, K)
    out = np.empty((rows, K), dtype=np.uint16)
    _check(lib().pqo_fakequant_int(_ptr(T), rows, K, K, bits, group, _ptr(perm), _ptr(out), K),
           "fakequant_int")
    return out


def gemm_ref(xq, sfx, ts_x, wq, sfw, ts_w):
    """fp64 product of the dequantized operands, [M, N]."""
    xq, sfx, wq, sfw = (np.ascontiguousarray(a, dtype=np.uint8) for a in (xq, sfx, wq, sfw))
    M, K = xq.shape[0], xq.shape[1] * 2
    N = wq.shape[0]
    Y = np.empty((M, N), dtype=np.float64)
    _check(lib().pqo_gemm_ref(_ptr(xq), _ptr(sfx), C.c_float(ts_x), _ptr(wq), _ptr(sfw),
                              C.c_float(ts_w), M, N, K, _ptr(Y)), "gemm_ref")
    return Y


def gemm_ref_sampled(xq, sfx, ts_x, wq, sfw, ts_w, ms, ns):
    """fp64 reference at the listed (m, n) entries only."""
    xq, sfx, wq, sfw = (np.ascontiguousarray(a, dtype=np.uint8) for a in (xq, sfx, wq, sfw))
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    K = xq.shape[1] * 2
    out = np.empty(ms.size, dtype=np.float64)
    _check(lib().pqo_gemm_ref_sampled(_ptr(xq), _ptr(sfx), C.c_float(ts_x), _ptr(wq), _ptr(sfw),
                                      C.c_float(ts_w), K, _ptr(ms), _ptr(ns), ms.size, _ptr(out)),
           "gemm_ref_sampled")
    return out


def gemm_bf16_ref(X, Wt, perm=None):
    """Unquantized fp64 product sum_k X[m, perm[k]] * Wt[n, perm[k]] (left side of Eq. 8)."""
    X, Wt = _bf16(X), _bf16(Wt)
    M, K = X.shape
    N = Wt.shape[0]
    perm = _perm(perm, K)
    Y = np.empty((M, N), dtype=np.float64)
    _check(lib().pqo_gemm_bf16_ref(_ptr(X), _ptr(Wt), M, N, K, _ptr(perm), _ptr(Y)), "gemm_bf16_ref")
    return Y


def chunk_rows():
    return int(lib().pqo_chunk_rows())


def slab_rows():
    return int(lib().pqo_slab_rows())
