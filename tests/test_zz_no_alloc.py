"""The workspace-free entry point against the ordinary one.

hif8_amax_scale_encode_static serves callers that may not allocate device memory where they call (code living
inside someone else's memory pool, latency-critical paths, fully pre-budgeted processes).  It must give exactly
what hif8_amax_scale_encode gives, also when called repeatedly: its scratch is one array inside the library that
keeps whatever the previous call left there.
"""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

pytestmark = pytest.mark.gpu


ORACLE_MODE = {H.RND_TA: O.TA, H.RND_HR: O.HR}


def run_both(src, dtype, target, mode, d_se_in=None):
    n = src.numel()
    wsb = H.hif8_workspace_bytes(H.WS_AMAX_SCALE_ENCODE, n)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    ref_codes = torch.empty(n, dtype=torch.uint8, device="cuda")
    ref_out = torch.zeros(4, dtype=torch.int32, device="cuda")
    H.hif8_amax_scale_encode(src, dtype, ref_codes, n, target, mode, 0, 3, d_se_in, ref_out[0:1], ref_out[1:2],
                             ref_out[2:3], ws, wsb)
    results = []
    for _ in range(2):                                   # two calls in a row share the library's scratch
        codes = torch.full((n,), 0xA5, dtype=torch.uint8, device="cuda")
        out = torch.zeros(4, dtype=torch.int32, device="cuda")
        H.hif8_amax_scale_encode_static(src, dtype, codes, n, target, mode, 0, 3, d_se_in, out[0:1], out[1:2], out[2:3])
        results.append((codes, out))
    torch.cuda.synchronize()
    # what the method defines, from the CPU oracle: amax over the tensor, the scale exponent, the codes
    host = src.cpu().numpy()
    host = host.view(np.uint16) if dtype != H.F32 else host
    amax, se = O.amax_scale(host, dtype, target)
    if d_se_in is not None:
        se = int(d_se_in.item())
    want = O.encode(host, dtype, se, ORACLE_MODE[mode], 0, seed=3, quick=True)
    for codes, out in results:
        assert torch.equal(codes, ref_codes)             # bit-exact, like every conversion test here
        assert torch.equal(out, ref_out)
        assert np.array_equal(codes.cpu().numpy(), want)
        o = out.cpu().numpy()
        assert o[0:1].view(np.float32)[0] == np.float32(amax) and int(o[1]) == se
        assert o[2:3].view(np.float32)[0] == np.float32(2.0 ** se)


def test_static_scratch_matches_workspace_variant():
    big = torch.from_numpy(W.normal_f32(1_000_003, seed=31)).cuda()
    small = torch.from_numpy(W.normal_f32(4099, seed=32) * np.float32(1e-3)).cuda()   # much smaller amax afterwards
    b16 = torch.from_numpy(W.normal_bf16(300_001, seed=33).view(np.int16)).cuda()
    run_both(big, H.F32, 14, H.RND_TA)
    run_both(small, H.F32, 14, H.RND_TA)                 # a stale maximum from `big` would change the scale
    run_both(b16, H.BF16, 3, H.RND_HR)
    d_se = torch.tensor([4], dtype=torch.int32, device="cuda")
    run_both(big, H.F32, 14, H.RND_TA, d_se)             # delayed-scaling form: amax still reduced through the scratch


def test_static_rejects_oversize_and_bad_arguments():
    before = H.hif8_launch_count()
    assert H.hif8_amax_scale_encode_static(0, H.F32, 0, (1 << 32) + 1, check=False) == 6
    assert H.hif8_amax_scale_encode_static(0, 9, 0, 16, check=False) == 2
    assert H.hif8_amax_scale_encode_static(0, H.F32, 0, 16, check=False) == 1
    assert H.hif8_launch_count() == before
