"""GPU side of the sharded per-tensor scaling path: hif8_amax + hif8_encode_from_amax through the C ABI, driven by
sharded.py under an NCCL process group of the one GPU this run provides, and with an amax planted as another rank's
all-reduce result would leave it."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O
from paper_2409_16626_b200 import sharded

from gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,rnd", [(H.F32, H.RND_TA), (H.BF16, H.RND_HR), (H.F16, H.RND_TA)])
def test_encode_from_amax_matches_oracle_for_a_foreign_amax(dtype, rnd):
    n = 300007
    x = W.normal_f32(n, 9)
    src = x if dtype == H.F32 else (W.f32_to_bf16_bits(x) if dtype == H.BF16 else x.astype(np.float16).view(np.uint16))
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    d_se = torch.zeros(1, dtype=torch.int32, device="cuda")
    d_scale = torch.zeros(1, dtype=torch.float32, device="cuda")
    for amax in (0.0, 1.0, 777.25, 3.0e-5, float(np.float32(2.0 ** -130)), 6.0e4):
        d_amax = torch.tensor([amax], dtype=torch.float32, device="cuda")
        H.hif8_encode_from_amax(to_dev(src), dtype, out, n, 9, rnd, 0, 0, d_amax, d_se, d_scale)
        se = O.amax_scale(np.array([amax], dtype=np.float32), O.F32, 9)[1]   # the per-tensor rule on that amax
        assert int(d_se.cpu()[0]) == se and float(d_scale.cpu()[0]) == 2.0 ** se
        assert np.array_equal(out.cpu().numpy(), O.encode(src, dtype, se, rnd, quick=True))
    assert H.hif8_encode_from_amax(to_dev(src), dtype, out, n, 9, rnd, 0, 0, None, check=False) == 1
    assert H.hif8_encode_from_amax(to_dev(src), dtype, out, n, 16, rnd, 0, 0, d_amax, check=False) == 5


def test_sharded_path_under_nccl_equals_the_just_in_time_call():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(33000 + os.getpid() % 2000))
    started = not dist.is_initialized()
    if started:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        n = 1 << 20
        x = W.normal_f32(n, 4)
        dx = to_dev(x)
        ws = torch.empty(256, dtype=torch.uint8, device="cuda")
        a = torch.empty(n, dtype=torch.uint8, device="cuda")
        b = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        d_se = torch.zeros(2, dtype=torch.int32, device="cuda")
        sharded.sharded_amax_scale_encode(H, dx, H.F32, a, n, 14, H.RND_TA, 0, 0, d_amax, ws, 256, d_se[0:1])
        H.hif8_amax_scale_encode(dx, H.F32, b, n, 14, H.RND_TA, 0, 0, None, None, d_se[1:2], None, ws, 256)
        amax, se = O.amax_scale(x, O.F32, 14)
        assert float(d_amax.cpu()[0]) == amax and d_se.cpu().tolist() == [se, se]
        assert torch.equal(a, b) and np.array_equal(a.cpu().numpy(), O.encode(x, O.F32, se, O.TA, quick=True))
    finally:
        if started:
            dist.destroy_process_group()
