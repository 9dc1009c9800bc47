"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and rejects bad
arguments before touching a device."""
import ctypes
import os
import re

import paper_2409_16626_b200 as H

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hif8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hif8_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(H.LIB_PATH)
    names = declared_symbols()
    assert {"hif8_encode", "hif8_decode", "hif8_amax_scale_encode", "hif8_fake_quant", "hif8_gemm"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_workspace():
    for s in range(0, 12):
        assert H.hif8_status_string(s) not in ("", "unknown status")
    assert H.hif8_status_string(99) == "unknown status"
    assert H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE, 1 << 20) >= 8
    assert H.hif8_workspace_bytes(H.WS_FAKE_QUANT, 1 << 20) >= 8


def test_argument_errors_before_any_launch():
    before = H.hif8_launch_count()
    assert H.hif8_encode(0, 7, 0, 16, stream=0, check=False) == 2            # dtype
    assert H.hif8_encode(0, H.F32, 0, 16, rnd=9, stream=0, check=False) == 3  # rounding
    assert H.hif8_encode(0, H.F32, 0, 16, flags=8, stream=0, check=False) == 4
    assert H.hif8_encode(0, H.F32, 0, 16, scale_exp=127, stream=0, check=False) == 5
    assert H.hif8_encode(0, H.F32, 0, 0, stream=0, check=False) == 0         # empty tensor is fine
    assert H.hif8_encode_f32_patterns(0, 0, 16, rnd=9, stream=0, check=False) == 3
    assert H.hif8_encode_f32_patterns(0, 0, (1 << 32) + 1, stream=0, check=False) == 6
    assert H.hif8_encode_f32_patterns(0, 0, 16, stream=0, check=False) == 1
    assert H.hif8_encode_f32_patterns(0, 0, 0, stream=0, check=False) == 0
    assert H.hif8_decode(0, 0, 5, 16, stream=0, check=False) == 2
    assert H.hif8_decode(0, 0, H.F16, 16, scale_exp=-127, stream=0, check=False) == 5
    assert H.hif8_decode(0, 0, H.F16, 0, stream=0, check=False) == 0
    assert H.hif8_amax_scale_encode(0, H.F32, 0, 16, target_exp=16, stream=0, check=False) == 5
    assert H.hif8_amax_scale_encode(0, H.F32, 0, 16, target_exp=14, stream=0, check=False) == 8   # no workspace
    assert H.hif8_fake_quant(0, 0, H.BF16, 16, use_amax=1, scale_or_target_exp=14, stream=0, check=False) == 8
    assert H.hif8_fake_quant(0, 0, H.BF16, 16, use_amax=0, scale_or_target_exp=200, stream=0, check=False) == 5
    assert H.hif8_launch_count() == before


def test_overlapping_source_and_destination_are_rejected_on_the_host():
    # a conversion reads one tensor and writes another; ranges that share a byte are refused before any launch
    before = H.hif8_launch_count()
    base = 1 << 20
    n = 1000
    assert H.hif8_encode(base, H.F32, base + 1, n, stream=0, check=False) == 11
    assert H.hif8_encode(base, H.F32, base + 4 * n - 1, n, stream=0, check=False) == 11      # last source byte
    assert H.hif8_encode(base + n - 1, H.BF16, base, n, stream=0, check=False) == 11         # destination ends inside
    assert H.hif8_decode(base, base + n - 1, H.F16, n, stream=0, check=False) == 11
    assert H.hif8_decode(base + 2 * n - 1, base, H.BF16, n, stream=0, check=False) == 11
    assert H.hif8_fake_quant(base, base + 2, H.BF16, n, use_amax=0, scale_or_target_exp=3, stream=0, check=False) == 11
    assert H.hif8_fake_quant(base + 4 * n - 4, base, H.F32, n, use_amax=0, scale_or_target_exp=3, stream=0, check=False) == 11
    assert H.hif8_amax_scale_encode(base, H.F32, base + 8, n, workspace=4096, workspace_bytes=256, stream=0, check=False) == 11
    assert H.hif8_amax_scale_encode_static(base, H.F32, base + 8, n, stream=0, check=False) == 11
    assert H.hif8_encode_from_amax(base, H.F16, base + 2 * n - 1, n, 14, H.RND_TA, 0, 0, 4096, stream=0, check=False) == 11
    assert H.hif8_encode_transpose(base, H.BF16, base + 100, 10, 100, stream=0, check=False) == 11
    assert H.hif8_channel_amax_scale_encode(base, H.BF16, base + 100, 10, 100, 0, d_amax=4096, stream=0, check=False) == 11
    assert H.hif8_launch_count() == before
    assert H.hif8_status_string(11) == "source and destination share bytes"


def test_host_side_caches_selftest():
    # the per-device set-up record (kernel attributes, SM count) and the tensor-map cache, driven without a device
    assert H.hif8_selftest_host_caches() == (0, 0)


def test_gemm_argument_errors_before_any_launch():
    before = H.hif8_launch_count()
    g = lambda **kw: H.hif8_gemm(kw.get("A", 16), kw.get("lda", 64), kw.get("W", 16), kw.get("ldw", 64), 0, kw.get("C", 16),
                                 kw.get("ldc", 64), kw.get("cdt", H.F32), kw.get("M", 64), kw.get("N", 64), kw.get("K", 64),
                                 None, None, kw.get("ws", 256), kw.get("wsb", 256), stream=0, check=False)
    assert g(cdt=H.F16) == 2
    assert g(K=40) == 6 and g(K=0) == 6 and g(M=-1) == 6 and g(lda=32) == 6 and g(ldc=32) == 6
    assert g(A=0) == 1
    assert g(A=24) == 7 and g(ldw=72) == 7 and g(ldc=66) == 7
    assert g(ws=0) == 8 and g(wsb=8) == 8
    assert g(M=0) == 0
    assert H.hif8_workspace_bytes(H.WS_GEMM) == 256
    assert H.hif8_launch_count() == before


def test_gemm_path_policy_setting_round_trips():
    # host-only: the setting is a process-wide integer; unknown values are refused and leave it alone
    before = H.hif8_gemm_path_policy(H.GEMM_PATH_EXPAND_BOTH)
    assert before in (H.GEMM_PATH_AUTO, H.GEMM_PATH_EXPAND_BOTH)
    assert H.hif8_gemm_path_policy(7) == 4                   # HIF8_ERR_FLAGS
    assert H.hif8_gemm_path_policy(H.GEMM_PATH_AUTO) == H.GEMM_PATH_EXPAND_BOTH
    assert H.hif8_gemm_path_policy(before) == H.GEMM_PATH_AUTO
