"""ctypes binding of libhif8.so.  Argument marshalling only: every step runs in the CUDA kernels.

Functions carry the C names and argument order of include/hif8.h.  Tensors are torch CUDA tensors (used for
device memory and streams only); pointers may also be given as plain ints.  A missing or unloadable library
is an error: there is no fallback path.
"""
import ctypes as C
import os

import torch

F32, BF16, F16 = 0, 1, 2
RND_TA, RND_HR, RND_SSR, RND_TE, RND_SR = 0, 1, 2, 3, 4
FLAG_SATURATE, FLAG_NAN_TO_ZERO = 1, 2
WS_AMAX_SCALE_ENCODE, WS_FAKE_QUANT, WS_GEMM = 0, 1, 2
OK = 0
SCALE_STATE_BYTES, SCALE_HISTORY_MAX = 1024, 32
ALS_STATE_BYTES = 64

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhif8.so")
EXPORTS = ["hif8_encode", "hif8_decode", "hif8_amax", "hif8_amax_scale_encode", "hif8_fake_quant", "hif8_gemm", "hif8_gemm_status", "hif8_pts_search", "hif8_pts_workspace_bytes",
           "hif8_pts_status", "hif8_selftest_wait_timeout", "hif8_channel_amax_scale_encode", "hif8_gemm_channel_scaled",
           "hif8_scale_state_init", "hif8_delayed_scale_encode", "hif8_gemm_ex", "hif8_encode_transpose", "hif8_als_state_init", "hif8_als_update", "hif8_check_finite", "hif8_encode_from_amax",
           "hif8_amax_scale_encode_static", "hif8_encode_f32_patterns", "hif8_last_device_status", "hif8_selftest_host_caches", "hif8_gemm_path_policy", "hif8_workspace_bytes", "hif8_status_string", "hif8_launch_count"]

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2409_16626_b200.build` (needs nvcc)")
lib = C.CDLL(LIB_PATH)

_vp, _sz, _i, _u, _u64, _i64 = C.c_void_p, C.c_size_t, C.c_int, C.c_uint, C.c_uint64, C.c_int64
lib.hif8_encode.argtypes = [_vp, _i, _vp, _sz, _i, _i, _u, _u64, _vp]
lib.hif8_decode.argtypes = [_vp, _vp, _i, _sz, _i, _vp]
lib.hif8_encode_f32_patterns.argtypes = [C.c_uint32, _vp, _sz, _i, _i, _u, _u64, _vp]
lib.hif8_encode_f32_patterns.restype = _i
lib.hif8_amax_scale_encode.argtypes = [_vp, _i, _vp, _sz, _i, _i, _u, _u64, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.hif8_amax.argtypes = [_vp, _i, _sz, _vp, _vp, _sz, _vp]
lib.hif8_amax.restype = _i
lib.hif8_amax_scale_encode_static.argtypes = [_vp, _i, _vp, _sz, _i, _i, _u, _u64, _vp, _vp, _vp, _vp, _vp]
lib.hif8_amax_scale_encode_static.restype = _i
lib.hif8_fake_quant.argtypes = [_vp, _vp, _i, _sz, _i, _i, _i, _u, _u64, _vp, _vp, _vp, _sz, _vp]
lib.hif8_gemm.argtypes = [_vp, _i64, _vp, _i64, _i, _vp, _i64, _i, _i, _i, _i, _vp, _vp, _vp, _sz, _vp]
lib.hif8_gemm_status.argtypes = [_vp, _vp]
lib.hif8_gemm_status.restype = _i
lib.hif8_gemm_path_policy.argtypes = [_i]
lib.hif8_gemm_path_policy.restype = _i
lib.hif8_pts_search.argtypes = [_vp, _vp, _i, _i, _vp, _i64, _i, _i, _i, _i, _i, _vp, _vp, _vp, _sz, _vp]
lib.hif8_pts_search.restype = _i
lib.hif8_pts_workspace_bytes.argtypes = [_i, _i, _i, _i]
lib.hif8_pts_workspace_bytes.restype = _sz
lib.hif8_pts_status.argtypes = [_vp, _vp]
lib.hif8_pts_status.restype = _i
lib.hif8_last_device_status.argtypes = [_vp]
lib.hif8_last_device_status.restype = _i
lib.hif8_selftest_host_caches.argtypes = [_vp]
lib.hif8_selftest_host_caches.restype = _i
lib.hif8_selftest_wait_timeout.argtypes = [_vp, _u, _vp]
lib.hif8_selftest_wait_timeout.restype = _i
lib.hif8_channel_amax_scale_encode.argtypes = [_vp, _i, _vp, _i64, _i64, _i, _i, _i, _u, _u64, _vp, _vp, _vp, _vp]
lib.hif8_channel_amax_scale_encode.restype = _i
lib.hif8_gemm_channel_scaled.argtypes = lib.hif8_gemm.argtypes
lib.hif8_gemm_channel_scaled.restype = _i
lib.hif8_scale_state_init.argtypes = [_vp, _i, _vp]
lib.hif8_scale_state_init.restype = _i
lib.hif8_delayed_scale_encode.argtypes = [_vp, _i, _vp, _sz, _i, _u, _u64, _vp, _i, _i, _vp]
lib.hif8_delayed_scale_encode.restype = _i
lib.hif8_gemm_ex.argtypes = [_vp, _i64, _i, _vp, _i64, _i, _vp, _i64, _i, _i, _i, _i, _vp, _vp, _vp, _i, _vp, _sz, _vp]
lib.hif8_gemm_ex.restype = _i
lib.hif8_encode_transpose.argtypes = [_vp, _i, _vp, _i64, _i64, _i, _vp, _i, _u, _u64, _vp]
lib.hif8_encode_transpose.restype = _i
lib.hif8_als_state_init.argtypes = [_vp, _i, _i, _vp]
lib.hif8_als_state_init.restype = _i
lib.hif8_als_update.argtypes = [_vp, _vp, _vp]
lib.hif8_als_update.restype = _i
lib.hif8_check_finite.argtypes = [_vp, _i, _sz, _vp, _vp]
lib.hif8_check_finite.restype = _i
lib.hif8_encode_from_amax.argtypes = [_vp, _i, _vp, _sz, _i, _i, _u, _u64, _vp, _vp, _vp, _vp]
lib.hif8_encode_from_amax.restype = _i
lib.hif8_workspace_bytes.argtypes = [_i, _sz]
lib.hif8_workspace_bytes.restype = _sz
lib.hif8_status_string.argtypes = [_i]
lib.hif8_status_string.restype = C.c_char_p
lib.hif8_launch_count.restype = _u64
for _n in ("hif8_encode", "hif8_decode", "hif8_amax_scale_encode", "hif8_fake_quant", "hif8_gemm"):
    getattr(lib, _n).restype = _i


class Hif8Error(RuntimeError):
    def __init__(self, status):
        self.status = status
        super().__init__(f"hif8 status {status}: {hif8_status_string(status)}")


def _ptr(t):
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


def _check(rc, check):
    if check and rc != OK:
        raise Hif8Error(rc)
    return rc


def hif8_status_string(status):
    return lib.hif8_status_string(int(status)).decode()


def hif8_workspace_bytes(which, n=0):
    return int(lib.hif8_workspace_bytes(which, n))


def hif8_launch_count():
    return int(lib.hif8_launch_count())


def hif8_encode(src, src_dtype, dst, n, scale_exp=0, rnd=RND_TA, flags=0, seed=0, stream=None, check=True):
    return _check(lib.hif8_encode(_ptr(src), src_dtype, _ptr(dst), n, scale_exp, rnd, flags, seed, _stream(stream)), check)


def hif8_encode_f32_patterns(first_pattern, dst, n, scale_exp=0, rnd=RND_TA, flags=0, seed=0, stream=None, check=True):
    return _check(lib.hif8_encode_f32_patterns(int(first_pattern) & 0xFFFFFFFF, _ptr(dst), n, scale_exp, rnd, flags, seed,
                                               _stream(stream)), check)


def hif8_decode(src, dst, dst_dtype, n, scale_exp=0, stream=None, check=True):
    return _check(lib.hif8_decode(_ptr(src), _ptr(dst), dst_dtype, n, scale_exp, _stream(stream)), check)


def hif8_amax_scale_encode(src, src_dtype, dst, n, target_exp=14, rnd=RND_TA, flags=0, seed=0, d_scale_exp_in=None,
                           d_amax_out=None, d_scale_exp_out=None, d_scale_out=None, workspace=None,
                           workspace_bytes=0, stream=None, check=True):
    return _check(lib.hif8_amax_scale_encode(_ptr(src), src_dtype, _ptr(dst), n, target_exp, rnd, flags, seed,
                                             _ptr(d_scale_exp_in), _ptr(d_amax_out), _ptr(d_scale_exp_out),
                                             _ptr(d_scale_out), _ptr(workspace), workspace_bytes, _stream(stream)), check)


def hif8_amax(src, src_dtype, n, d_amax_out, workspace, workspace_bytes, stream=None, check=True):
    return _check(lib.hif8_amax(_ptr(src), src_dtype, n, _ptr(d_amax_out), _ptr(workspace), workspace_bytes, _stream(stream)), check)


def hif8_amax_scale_encode_static(src, src_dtype, dst, n, target_exp=14, rnd=RND_TA, flags=0, seed=0,
                                  d_scale_exp_in=None, d_amax_out=None, d_scale_exp_out=None, d_scale_out=None,
                                  stream=None, check=True):
    """hif8_amax_scale_encode for callers that cannot hand over a workspace (scratch lives inside the library)."""
    return _check(lib.hif8_amax_scale_encode_static(_ptr(src), src_dtype, _ptr(dst), n, target_exp, rnd, flags, seed,
                                                    _ptr(d_scale_exp_in), _ptr(d_amax_out), _ptr(d_scale_exp_out),
                                                    _ptr(d_scale_out), _stream(stream)), check)


def hif8_fake_quant(src, dst, dtype, n, use_amax=0, scale_or_target_exp=0, rnd=RND_TA, flags=0, seed=0,
                    d_amax_out=None, d_scale_exp_out=None, workspace=None, workspace_bytes=0, stream=None, check=True):
    return _check(lib.hif8_fake_quant(_ptr(src), _ptr(dst), dtype, n, use_amax, scale_or_target_exp, rnd, flags, seed,
                                      _ptr(d_amax_out), _ptr(d_scale_exp_out), _ptr(workspace), workspace_bytes,
                                      _stream(stream)), check)


def hif8_gemm(Aq, lda, Wq, ldw, w_is_nk, Cmat, ldc, c_dtype, M, N, K, d_scale_exp_a=None, d_scale_exp_w=None,
              workspace=None, workspace_bytes=0, stream=None, check=True):
    return _check(lib.hif8_gemm(_ptr(Aq), lda, _ptr(Wq), ldw, w_is_nk, _ptr(Cmat), ldc, c_dtype, M, N, K,
                                _ptr(d_scale_exp_a), _ptr(d_scale_exp_w), _ptr(workspace), workspace_bytes,
                                _stream(stream)), check)


def hif8_gemm_status(workspace, stream=None):
    return int(lib.hif8_gemm_status(_ptr(workspace), _stream(stream)))


GEMM_PATH_AUTO, GEMM_PATH_EXPAND_BOTH = 0, 1


def hif8_gemm_path_policy(policy):
    """Sets which general kernel a large workspace selects; returns the previous setting, or 4 (HIF8_ERR_FLAGS) for an unknown one."""
    return int(lib.hif8_gemm_path_policy(int(policy)))


def hif8_pts_workspace_bytes(M, N, K, n_exp):
    return int(lib.hif8_pts_workspace_bytes(M, N, K, n_exp))


def hif8_pts_search(A, W, dtype, w_is_nk, O_ref, ldo, M, N, K, e_min, e_max, d_err, d_best, workspace, workspace_bytes,
                    stream=None, check=True):
    return _check(lib.hif8_pts_search(_ptr(A), _ptr(W), dtype, int(w_is_nk), _ptr(O_ref), ldo, M, N, K, e_min, e_max,
                                      _ptr(d_err), _ptr(d_best), _ptr(workspace), workspace_bytes, _stream(stream)), check)


def hif8_pts_status(workspace, stream=None):
    return int(lib.hif8_pts_status(_ptr(workspace), _stream(stream)))


def hif8_last_device_status(stream=None):
    return int(lib.hif8_last_device_status(_stream(stream)))


def hif8_selftest_host_caches():
    """(status, number of the failed check or 0)"""
    failed = C.c_int(-1)
    rc = int(lib.hif8_selftest_host_caches(C.byref(failed)))
    return rc, int(failed.value)


def hif8_selftest_wait_timeout(workspace, limit_ms, stream=None, check=True):
    return _check(lib.hif8_selftest_wait_timeout(_ptr(workspace), limit_ms, _stream(stream)), check)


def hif8_channel_amax_scale_encode(W, src_dtype, dst, rows, cols, channel_axis, target_exp=14, rnd=RND_TA, flags=0, seed=0,
                                   d_scale_exp_in=None, d_amax=None, d_scale_exp_out=None, stream=None, check=True):
    return _check(lib.hif8_channel_amax_scale_encode(_ptr(W), src_dtype, _ptr(dst), rows, cols, channel_axis, target_exp, rnd,
                                                     flags, seed, _ptr(d_scale_exp_in), _ptr(d_amax), _ptr(d_scale_exp_out),
                                                     _stream(stream)), check)


def hif8_gemm_channel_scaled(Aq, lda, Wq, ldw, w_is_nk, Cmat, ldc, c_dtype, M, N, K, d_scale_exp_a=None,
                             d_scale_exp_w_channel=None, workspace=None, workspace_bytes=0, stream=None, check=True):
    return _check(lib.hif8_gemm_channel_scaled(_ptr(Aq), lda, _ptr(Wq), ldw, w_is_nk, _ptr(Cmat), ldc, c_dtype, M, N, K,
                                               _ptr(d_scale_exp_a), _ptr(d_scale_exp_w_channel), _ptr(workspace),
                                               workspace_bytes, _stream(stream)), check)


def hif8_scale_state_init(d_state, hist_len, stream=None, check=True):
    return _check(lib.hif8_scale_state_init(_ptr(d_state), hist_len, _stream(stream)), check)


def hif8_delayed_scale_encode(src, src_dtype, dst, n, rnd, flags, seed, d_state, measure, target_exp=14, stream=None,
                              check=True):
    return _check(lib.hif8_delayed_scale_encode(_ptr(src), src_dtype, _ptr(dst), n, rnd, flags, seed, _ptr(d_state),
                                                int(measure), target_exp, _stream(stream)), check)


def hif8_gemm_ex(Aq, lda, a_is_km, Wq, ldw, w_is_nk, Cmat, ldc, c_dtype, M, N, K, d_scale_exp_a=None, d_scale_exp_w=None,
                 d_scale_exp_w_channel=None, accumulate=0, workspace=None, workspace_bytes=0, stream=None, check=True):
    return _check(lib.hif8_gemm_ex(_ptr(Aq), lda, int(a_is_km), _ptr(Wq), ldw, int(w_is_nk), _ptr(Cmat), ldc, c_dtype, M, N, K,
                                   _ptr(d_scale_exp_a), _ptr(d_scale_exp_w), _ptr(d_scale_exp_w_channel), int(accumulate),
                                   _ptr(workspace), workspace_bytes, _stream(stream)), check)


def hif8_encode_transpose(src, src_dtype, dst, rows, cols, scale_exp=0, d_scale_exp=None, rnd=RND_TA, flags=0, seed=0,
                          stream=None, check=True):
    return _check(lib.hif8_encode_transpose(_ptr(src), src_dtype, _ptr(dst), rows, cols, scale_exp, _ptr(d_scale_exp), rnd,
                                            flags, seed, _stream(stream)), check)


def hif8_als_state_init(d_state, init_scale_exp=32, init_window_index=1, stream=None, check=True):
    return _check(lib.hif8_als_state_init(_ptr(d_state), init_scale_exp, init_window_index, _stream(stream)), check)


def hif8_als_update(d_state, d_found_inf, stream=None, check=True):
    return _check(lib.hif8_als_update(_ptr(d_state), _ptr(d_found_inf), _stream(stream)), check)


def hif8_check_finite(src, dtype, n, d_found_inf, stream=None, check=True):
    return _check(lib.hif8_check_finite(_ptr(src), dtype, n, _ptr(d_found_inf), _stream(stream)), check)


def hif8_encode_from_amax(src, src_dtype, dst, n, target_exp, rnd, flags, seed, d_amax, d_scale_exp_out=None, d_scale_out=None,
                          stream=None, check=True):
    return _check(lib.hif8_encode_from_amax(_ptr(src), src_dtype, _ptr(dst), n, target_exp, rnd, flags, seed, _ptr(d_amax),
                                            _ptr(d_scale_exp_out), _ptr(d_scale_out), _stream(stream)), check)
