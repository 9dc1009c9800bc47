"""Helpers for the GPU parity tests: raw-bit numpy arrays <-> device buffers."""
import numpy as np
import torch

import paper_2409_16626_b200 as H

NP_OF = {H.F32: np.uint32, H.BF16: np.uint16, H.F16: np.uint16}


def to_dev(a):
    """numpy array of raw encodings -> CUDA tensor with the same bytes."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        a = a.view(np.uint32)
    signed = {np.dtype(np.uint8): np.uint8, np.dtype(np.uint16): np.int16, np.dtype(np.uint32): np.int32}[a.dtype]
    return torch.from_numpy(a.view(signed)).cuda()


def dev_empty(n, np_dtype, offset_bytes=0):
    """n elements of np_dtype on the device, optionally starting `offset_bytes` into a 256-byte aligned buffer.
    Returns (tensor-owner, pointer, readback) where readback() gives a numpy array of raw encodings."""
    item = np.dtype(np_dtype).itemsize
    raw = torch.empty(n * item + offset_bytes + 64, dtype=torch.uint8, device="cuda")
    raw.fill_(0xA5)
    ptr = raw.data_ptr() + offset_bytes

    def readback():
        b = raw.cpu().numpy()
        assert np.all(b[:offset_bytes] == 0xA5) and np.all(b[offset_bytes + n * item:] == 0xA5), "write outside the output"
        return b[offset_bytes:offset_bytes + n * item].copy().view(np_dtype)

    return raw, ptr, readback


def workspace():
    n = H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE)
    return torch.empty(max(n, 256), dtype=torch.uint8, device="cuda"), n


def bf16_half_ulp(x):
    """Half a unit in the last place of a bfloat16 (8-bit significand) at the binade of |x| (normal range):
    what one round-to-nearest into BF16 can cost."""
    e = np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -126)))
    return 2.0 ** (e - 8)


import contextlib


@contextlib.contextmanager
def both_operands_expanded(on):
    """Within the block a workspace with room for both operands selects the kernel that expands both, whatever the size of
    the product (hif8_gemm_path_policy); the previous setting is restored afterwards."""
    import paper_2409_16626_b200 as H
    before = H.hif8_gemm_path_policy(H.GEMM_PATH_EXPAND_BOTH if on else H.GEMM_PATH_AUTO)
    try:
        yield
    finally:
        H.hif8_gemm_path_policy(before)
