"""ctypes front end of the C oracle (oracle/hif8_oracle.c).

Test infrastructure: only tests/, the smoke check and the benchmark's CPU-baseline leg use it.
Arrays are numpy; 16-bit float formats travel as uint16 encodings, FP32 as float32 or uint32.
"""
import ctypes as C
import numpy as np

from . import build as _build

F32, BF16, F16 = 0, 1, 2
TA, HR, SSR, TE, SR = 0, 1, 2, 3, 4
SATURATE, NAN_TO_ZERO = 1, 2

_lib = C.CDLL(_build.build())
_vp, _sz, _i, _u, _u64, _ll = C.c_void_p, C.c_size_t, C.c_int, C.c_uint, C.c_uint64, C.c_longlong

_lib.hif8o_value.restype = C.c_double
_lib.hif8o_value.argtypes = [_u]
_lib.hif8o_parse.argtypes = [_u] + [C.POINTER(C.c_int)] * 7 + [C.POINTER(C.c_double)]
_lib.hif8o_round_to_format.restype = C.c_uint32
_lib.hif8o_round_to_format.argtypes = [C.c_double, _i, _i]
_lib.hif8o_sr_word.restype = C.c_uint32
_lib.hif8o_sr_word.argtypes = [_u64, _u64]
_lib.hif8o_philox4x32_10.argtypes = [_vp, _vp, _vp]
_lib.hif8o_num_threads.restype = _i
_lib.hif8o_encode.argtypes = [_vp, _i, _vp, _sz, _i, _i, _u, _u64, _i]
_lib.hif8o_encode_at.argtypes = [_vp, _i, _vp, _sz, _vp, _i, _i, _u, _u64, _i]
_lib.hif8o_fake_quant_at.argtypes = [_vp, _vp, _i, _sz, _vp, _i, _i, _u, _u64, _i]
_lib.hif8o_encode_f32_range.argtypes = [C.c_uint32, _sz, _vp, _i, _i, _u, _u64, _i]
_lib.hif8o_decode.argtypes = [_vp, _vp, _i, _sz, _i]
_lib.hif8o_amax_scale.argtypes = [_vp, _i, _sz, _i, C.POINTER(C.c_float), C.POINTER(C.c_int)]
_lib.hif8o_fake_quant.argtypes = [_vp, _vp, _i, _sz, _i, _i, _u, _u64, _i]
_lib.hif8o_gemm_entries.argtypes = [_vp, _ll, _vp, _ll, _i, _i, _i, _i, _vp, _vp, _sz, _vp, _vp]
_lib.hif8o_pts_search.argtypes = [_vp, _vp, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp]
_lib.hif8o_channel_amax_scale.argtypes = [_vp, _i, _ll, _ll, _i, _i, _vp, _vp]
_lib.hif8o_channel_encode.argtypes = [_vp, _i, _vp, _ll, _ll, _i, _vp, _i, _u, _u64, _i]
_lib.hif8o_gemm_entries_channel.argtypes = [_vp, _ll, _vp, _ll, _i, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.hif8o_delayed_scale_run.argtypes = [_vp, _i, _i, _i, _i, _vp]
_lib.hif8o_encode_transpose.argtypes = [_vp, _i, _vp, _ll, _ll, _i, _i, _u, _u64, _i]
_lib.hif8o_gemm_entries_ex.argtypes = [_vp, _ll, _i, _vp, _ll, _i, _i, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]
_lib.hif8o_als_run.argtypes = [_vp, _i, _i, _i, _vp, _vp]
_lib.hif8o_gemm_full.argtypes = [_vp, _ll, _vp, _ll, _i, _i, _i, _i, _i, _i, _vp, _vp]


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def _src(a, dtype):
    a = np.ascontiguousarray(a)
    if dtype == F32:
        assert a.dtype in (np.float32, np.uint32), a.dtype
    else:
        assert a.dtype == np.uint16, a.dtype
    return a


def _out_dtype(dtype):
    return np.uint32 if dtype == F32 else np.uint16


def num_threads():
    return int(_lib.hif8o_num_threads())


def value(code):
    """Real value of one byte (float: nan, +-inf, 0.0 or finite)."""
    return float(_lib.hif8o_value(int(code)))


def parse(code):
    """Fields of one byte: dict(kind, sign, is_dml, D, E, w, M, value); kind 0 zero, 1 finite, 2 inf, 3 nan.
    For the Inf patterns `value` is the Eq. 1 value +-1.5*2^15."""
    ints = [C.c_int() for _ in range(7)]
    v = C.c_double()
    _lib.hif8o_parse(int(code), *[C.byref(x) for x in ints], C.byref(v))
    names = ["kind", "sign", "is_dml", "D", "E", "w", "M"]
    d = {k: x.value for k, x in zip(names, ints)}
    d["value"] = v.value
    return d


def round_to_format(v, ebits, mbits):
    return int(_lib.hif8o_round_to_format(float(v), ebits, mbits))


def sr_word(seed, idx):
    return int(_lib.hif8o_sr_word(int(seed), int(idx)))


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    _lib.hif8o_philox4x32_10(_ptr(c), _ptr(k), _ptr(o))
    return o


def encode(src, dtype, scale_exp=0, rnd=TA, flags=0, seed=0, quick=False):
    a = _src(src, dtype)
    out = np.empty(a.size, dtype=np.uint8)
    _lib.hif8o_encode(_ptr(a), dtype, _ptr(out), a.size, scale_exp, rnd, flags, seed, int(quick))
    return out.reshape(a.shape)


def encode_at(src, dtype, idx, scale_exp=0, rnd=TA, flags=0, seed=0, quick=False):
    """Codes of elements taken out of a larger tensor: src[j] sat at flat position idx[j] (matters for SR only)."""
    a = _src(src, dtype)
    ix = np.ascontiguousarray(idx, dtype=np.uint64)
    assert ix.size == a.size
    out = np.empty(a.size, dtype=np.uint8)
    _lib.hif8o_encode_at(_ptr(a), dtype, _ptr(out), a.size, _ptr(ix), scale_exp, rnd, flags, seed, int(quick))
    return out.reshape(a.shape)


def fake_quant_at(src, dtype, idx, scale_exp=0, rnd=TA, flags=0, seed=0, quick=False):
    a = _src(src, dtype)
    ix = np.ascontiguousarray(idx, dtype=np.uint64)
    assert ix.size == a.size
    out = np.empty(a.size, dtype=_out_dtype(dtype))
    _lib.hif8o_fake_quant_at(_ptr(a), _ptr(out), dtype, a.size, _ptr(ix), scale_exp, rnd, flags, seed, int(quick))
    return out.reshape(a.shape)


def encode_f32_range(first, n, scale_exp=0, rnd=TA, flags=0, seed=0, quick=True):
    out = np.empty(n, dtype=np.uint8)
    _lib.hif8o_encode_f32_range(int(first) & 0xFFFFFFFF, n, _ptr(out), scale_exp, rnd, flags, seed, int(quick))
    return out


def decode(codes, dtype, scale_exp=0):
    a = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(a.size, dtype=_out_dtype(dtype))
    _lib.hif8o_decode(_ptr(a), _ptr(out), dtype, a.size, scale_exp)
    return out.reshape(a.shape)


def amax_scale(src, dtype, target_exp=14):
    a = _src(src, dtype)
    amax, se = C.c_float(), C.c_int()
    _lib.hif8o_amax_scale(_ptr(a), dtype, a.size, target_exp, C.byref(amax), C.byref(se))
    return float(amax.value), int(se.value)


def fake_quant(src, dtype, scale_exp=0, rnd=TA, flags=0, seed=0, quick=False):
    a = _src(src, dtype)
    out = np.empty(a.size, dtype=_out_dtype(dtype))
    _lib.hif8o_fake_quant(_ptr(a), _ptr(out), dtype, a.size, scale_exp, rnd, flags, seed, int(quick))
    return out.reshape(a.shape)


def gemm_entries(Aq, Wq, w_is_nk, sa, sw, rows, cols):
    """(C*, S) in float64 for the listed (row, col) entries; Aq [M,K], Wq [K,N] or [N,K] uint8."""
    Aq = np.ascontiguousarray(Aq, dtype=np.uint8)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    K = Aq.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    cs = np.empty(rows.size, dtype=np.float64)
    s = np.empty(rows.size, dtype=np.float64)
    _lib.hif8o_gemm_entries(_ptr(Aq), Aq.shape[1], _ptr(Wq), Wq.shape[1], int(w_is_nk), K, sa, sw,
                            _ptr(rows), _ptr(cols), rows.size, _ptr(cs), _ptr(s))
    return cs, s


def gemm_full(Aq, Wq, w_is_nk, sa, sw):
    Aq = np.ascontiguousarray(Aq, dtype=np.uint8)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    M, K = Aq.shape
    N = Wq.shape[0] if w_is_nk else Wq.shape[1]
    cs = np.empty((M, N), dtype=np.float64)
    s = np.empty((M, N), dtype=np.float64)
    _lib.hif8o_gemm_full(_ptr(Aq), K, _ptr(Wq), Wq.shape[1], int(w_is_nk), M, N, K, sa, sw, _ptr(cs), _ptr(s))
    return cs, s


def pts_search(A, W, dtype, w_is_nk, O_ref, e_min=-4, e_max=5, quick=False):
    """Algorithm 1 for one layer: (err[nE, nE] float64 MSE table indexed [Ea - e_min, Ew - e_min], (best Ea, best Ew)).
    A [M,K], W [K,N] or [N,K] raw encodings of `dtype`; O_ref [M,N] float32."""
    A = _src(A, dtype)
    W = _src(W, dtype)
    O_ref = np.ascontiguousarray(O_ref, dtype=np.float32)
    M, K = A.shape
    N = W.shape[0] if w_is_nk else W.shape[1]
    nE = e_max - e_min + 1
    err = np.empty((nE, nE), dtype=np.float64)
    best = np.zeros(2, dtype=np.int32)
    _lib.hif8o_pts_search(_ptr(A), _ptr(W), dtype, int(w_is_nk), _ptr(O_ref), M, N, K, e_min, e_max, int(quick),
                          _ptr(err), _ptr(best))
    return err, (int(best[0]), int(best[1]))


def channel_amax_scale(W, dtype, axis, target_exp=14):
    """Per-channel amax (float32) and scale exponents (int32) of W [rows, cols]; axis 0: channel = row, 1: column."""
    W = _src(W, dtype)
    rows, cols = W.shape
    ch = rows if axis == 0 else cols
    amax = np.empty(ch, dtype=np.float32)
    se = np.empty(ch, dtype=np.int32)
    _lib.hif8o_channel_amax_scale(_ptr(W), dtype, rows, cols, axis, target_exp, _ptr(amax), _ptr(se))
    return amax, se


def channel_encode(W, dtype, axis, scale_exp, rnd=TA, flags=0, seed=0, quick=False):
    W = _src(W, dtype)
    rows, cols = W.shape
    se = np.ascontiguousarray(scale_exp, dtype=np.int32)
    assert se.size == (rows if axis == 0 else cols)
    out = np.empty((rows, cols), dtype=np.uint8)
    _lib.hif8o_channel_encode(_ptr(W), dtype, _ptr(out), rows, cols, axis, _ptr(se), rnd, flags, seed, int(quick))
    return out


def gemm_entries_channel(Aq, Wq, w_is_nk, sa, sw, rows, cols):
    """As gemm_entries with one weight exponent per output column: sw int32 [N]."""
    Aq = np.ascontiguousarray(Aq, dtype=np.uint8)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    K = Aq.shape[1]
    sw = np.ascontiguousarray(sw, dtype=np.int32)
    assert sw.size == (Wq.shape[0] if w_is_nk else Wq.shape[1])
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    cs = np.empty(rows.size, dtype=np.float64)
    s = np.empty(rows.size, dtype=np.float64)
    _lib.hif8o_gemm_entries_channel(_ptr(Aq), Aq.shape[1], _ptr(Wq), Wq.shape[1], int(w_is_nk), K, sa, _ptr(sw),
                                    _ptr(rows), _ptr(cols), rows.size, _ptr(cs), _ptr(s))
    return cs, s


def delayed_scale_run(amax, interval, hist_len, target_exp=14):
    """Exponent in force at each iteration of the every-`interval`-iterations amax cadence (int32 [T])."""
    amax = np.ascontiguousarray(amax, dtype=np.float32)
    used = np.empty(amax.size, dtype=np.int32)
    _lib.hif8o_delayed_scale_run(_ptr(amax), amax.size, interval, hist_len, target_exp, _ptr(used))
    return used


def encode_transpose(src, dtype, scale_exp=0, rnd=TA, flags=0, seed=0, quick=False):
    """Codes of src [rows, cols], stored transposed: uint8 [cols, rows]."""
    a = _src(src, dtype)
    rows, cols = a.shape
    out = np.empty((cols, rows), dtype=np.uint8)
    _lib.hif8o_encode_transpose(_ptr(a), dtype, _ptr(out), rows, cols, scale_exp, rnd, flags, seed, int(quick))
    return out


def gemm_entries_ex(Aq, a_is_km, Wq, w_is_nk, sa, sw, rows, cols):
    """(C*, S) for listed entries; Aq [M,K] or (a_is_km) [K,M]; Wq [K,N] or (w_is_nk) [N,K]; sw an int or an int32 [N]."""
    Aq = np.ascontiguousarray(Aq, dtype=np.uint8)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    K = Aq.shape[0] if a_is_km else Aq.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    cs = np.empty(rows.size, dtype=np.float64)
    s = np.empty(rows.size, dtype=np.float64)
    ch = None if np.isscalar(sw) else np.ascontiguousarray(sw, dtype=np.int32)
    _lib.hif8o_gemm_entries_ex(_ptr(Aq), Aq.shape[1], int(a_is_km), _ptr(Wq), Wq.shape[1], int(w_is_nk), K, sa,
                               int(sw) if ch is None else 0, None if ch is None else _ptr(ch), _ptr(rows), _ptr(cols),
                               rows.size, _ptr(cs), _ptr(s))
    return cs, s


ALS_WINDOWS = (1, 20, 50, 100, 200, 500, 1000)


def als_run(found_inf, init_scale_exp=32, init_window_index=1):
    """Adaptive loss scaling over a sequence of overflow flags: (log2 scale, window) in force during each iteration."""
    f = np.ascontiguousarray(found_inf, dtype=np.int32)
    se = np.empty(f.size, dtype=np.int32)
    win = np.empty(f.size, dtype=np.int32)
    _lib.hif8o_als_run(_ptr(f), f.size, init_scale_exp, init_window_index, _ptr(se), _ptr(win))
    return se, win
