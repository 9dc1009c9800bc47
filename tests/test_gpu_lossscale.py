"""GPU parity (through the C ABI) of adaptive loss scaling (Section 5.1 ALS): the overflow check of gradient tensors
and the device-resident scale / window controller against the oracle's sequence state machine."""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import to_dev

pytestmark = pytest.mark.gpu


def as_dtype(x, dtype):
    if dtype == H.F32:
        return x
    if dtype == H.BF16:
        return W.f32_to_bf16_bits(x)
    with np.errstate(over="ignore"):
        return np.where(np.isfinite(x), np.clip(x, -65504, 65504), x).astype(np.float16).view(np.uint16)


@pytest.mark.parametrize("dtype", [H.F32, H.BF16, H.F16])
@pytest.mark.parametrize("n,offset", [(1 << 20, 0), (100003, 0), (4099, 1), (7, 0)])
def test_check_finite_finds_exactly_the_planted_specials(dtype, n, offset):
    item = 4 if dtype == H.F32 else 2
    x = W.loguniform_f32(n, 3).astype(np.float32)
    big = {H.F32: np.float32(3.4e38), H.BF16: np.float32(3.38e38), H.F16: np.float32(65504.0)}[dtype]
    x[n // 2] = big            # the largest finite value is not an overflow
    x[0] = -big
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run(arr):
        raw = np.ascontiguousarray(as_dtype(arr, dtype)).view(np.uint8)
        buf = torch.zeros(raw.size + 64, dtype=torch.uint8, device="cuda")
        buf[offset * item:offset * item + raw.size] = torch.from_numpy(raw.copy()).cuda()
        H.hif8_check_finite(buf.data_ptr() + offset * item, dtype, n, flag)
        return int(flag.cpu()[0])

    assert run(x) == 0
    for pos, val in ((0, np.inf), (n - 1, -np.inf), (n // 3, np.nan), (n - 1, np.nan)):
        y = x.copy()
        y[pos] = val
        flag.zero_()
        assert run(y) == 1, (pos, val)
    assert run(x) == 1          # the flag is sticky until the controller (or the caller) clears it
    flag.zero_()
    assert H.hif8_check_finite(None, dtype, 0, flag) == 0 and int(flag.cpu()[0]) == 0


def test_als_controller_follows_the_oracle_over_a_long_run():
    rng = np.random.default_rng(11)
    T = 1500
    f = (rng.random(T) < 0.03).astype(np.int32)
    f[200:203] = 1
    f[700:707] = 1
    se, win = O.als_run(f, 32, 1)
    state = torch.zeros(H.ALS_STATE_BYTES // 4, dtype=torch.int32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    H.hif8_als_state_init(state)
    clean = torch.ones(4096, dtype=torch.float32, device="cuda")
    dirty = clean.clone()
    dirty[1234] = float("inf")
    snaps = torch.zeros(T, 8, dtype=torch.int32, device="cuda")
    for t in range(T):
        snaps[t].copy_(state[:8])                            # the state in force during iteration t
        H.hif8_check_finite(dirty if f[t] else clean, H.F32, 4096, flag)
        H.hif8_als_update(state, flag)
    snaps = snaps.cpu().numpy()
    assert np.array_equal(snaps[:, 0], se) and np.array_equal(snaps[:, 1], win)
    assert np.array_equal(snaps[:, 6], np.arange(T)) and snaps[-1, 7] == f[:-1].sum()
    assert int(flag.cpu()[0]) == 0
    assert len(set(win.tolist())) >= 3


def test_als_gradient_pipeline_on_the_device():
    # scaled gradients overflow FP16 while the scale is too large; the controller halves it until they fit, with no
    # host decision in the loop: every iteration runs the same calls
    g = (W.normal_f32(1 << 16, 5) * np.float32(1e-3)).astype(np.float32)
    state = torch.zeros(16, dtype=torch.int32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    H.hif8_als_state_init(state, 32, 1)
    gd = torch.from_numpy(g).cuda()
    seen = []
    for it in range(40):
        s = state[0:1].float()                                  # loss scale exponent, read on the device
        scaled = (gd * torch.exp2(s)).to(torch.float16)        # stands in for a backward pass in FP16
        H.hif8_check_finite(scaled, H.F16, scaled.numel(), flag)
        H.hif8_als_update(state, flag)
        seen.append(int(state[0].cpu()))
    amax = float(np.abs(g).max())
    fits = int(np.floor(np.log2(65504.0 / amax)))
    assert seen[0] == 31 and min(seen) >= fits - 1 and seen[-1] <= fits + 1


def test_als_argument_checks():
    state = torch.zeros(16, dtype=torch.int32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert H.hif8_als_state_init(None, check=False) == 1
    assert H.hif8_als_state_init(state.data_ptr() + 4, check=False) == 7
    assert H.hif8_als_state_init(state, 127, 1, check=False) == 5
    assert H.hif8_als_state_init(state, 32, 7, check=False) == 6
    assert H.hif8_als_update(state, None, check=False) == 1
    assert H.hif8_check_finite(state, 9, 4, flag, check=False) == 2
    assert H.hif8_check_finite(state, H.F32, 4, None, check=False) == 1
    assert H.hif8_check_finite(state.data_ptr() + 2, H.F32, 2, flag, check=False) == 7
