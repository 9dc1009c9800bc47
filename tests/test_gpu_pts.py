"""GPU parity of hif8_pts_search (Algorithm 1, per-layer search) against the CPU oracle.

Tolerance: each MSE entry within 1e-4 relative (FP32 tensor-core accumulation of exact products vs FP64; the error
sum itself is accumulated in double on both sides).  The argmin must match unless the two best entries of the
oracle's table are closer than that tolerance."""
import numpy as np
import pytest
import torch

import paper_2409_16626_b200 as H
import workloads as W
from oracle import hif8_oracle as O

from gpu_util import to_dev

pytestmark = pytest.mark.gpu


def run(A, Wm, dtype, w_is_nk, Oref, e_min, e_max):
    M, K = A.shape
    N = Wm.shape[0] if w_is_nk else Wm.shape[1]
    n = e_max - e_min + 1
    wsb = H.hif8_pts_workspace_bytes(M, N, K, n)
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    d_err = torch.zeros(n * n, dtype=torch.float32, device="cuda")
    d_best = torch.zeros(2, dtype=torch.int32, device="cuda")
    dO = torch.from_numpy(Oref).cuda()
    H.hif8_pts_search(to_dev(A), to_dev(Wm), dtype, w_is_nk, dO, N, M, N, K, e_min, e_max, d_err, d_best, ws, wsb)
    assert H.hif8_pts_status(ws) == 0
    return d_err.cpu().numpy().reshape(n, n).astype(np.float64), tuple(int(v) for v in d_best.cpu())


@pytest.mark.parametrize("case", [(96, 160, 256, O.BF16, 0), (130, 272, 208, O.F32, 1), (256, 512, 512, O.BF16, 1)])
def test_pts_search_matches_oracle(case):
    M, N, K, dtype, w_is_nk = case
    if dtype == O.BF16:
        a, w = W.normal_bf16((M, K), seed=M), W.normal_bf16((K, N), seed=N, std=0.03)
        af, wf = W.bf16_bits_to_f32(a).astype(np.float64), W.bf16_bits_to_f32(w).astype(np.float64)
    else:
        a32, w32 = W.normal_f32((M, K), seed=M), W.normal_f32((K, N), seed=N, std=0.03)
        a, w = a32.view(np.uint32), w32.view(np.uint32)
        af, wf = a32.astype(np.float64), w32.astype(np.float64)
    Oref = (af @ wf).astype(np.float32)
    wm = np.ascontiguousarray(w.T) if w_is_nk else w
    want, best = O.pts_search(a, wm, dtype, w_is_nk, Oref, -4, 5, quick=True)
    got, gbest = run(a, wm, dtype, w_is_nk, Oref, -4, 5)
    assert np.allclose(got, want, rtol=1e-4, atol=0), np.max(np.abs(got / want - 1))
    srt = np.sort(want.ravel())
    if srt[1] / srt[0] - 1 > 2e-4:
        assert gbest == best
    else:
        assert want[gbest[0] + 4, gbest[1] + 4] <= srt[0] * (1 + 2e-4)


def test_pts_search_small_grid_and_arguments():
    M, N, K = 64, 64, 64
    a, w = W.normal_bf16((M, K), seed=1), W.normal_bf16((K, N), seed=2)
    Oref = (W.bf16_bits_to_f32(a).astype(np.float64) @ W.bf16_bits_to_f32(w).astype(np.float64)).astype(np.float32)
    want, best = O.pts_search(a, w, O.BF16, False, Oref, 0, 1)
    got, gbest = run(a, w, O.BF16, 0, Oref, 0, 1)
    assert np.allclose(got, want, rtol=1e-4) and gbest == best
    assert H.hif8_pts_search(16, 16, H.BF16, 0, 16, N, M, N, K, -4, 20, 16, 16, 256, 1 << 30, check=False) == 5
    assert H.hif8_pts_search(16, 16, H.BF16, 0, 16, N, M, N, 40, -4, 5, 16, 16, 256, 1 << 30, check=False) == 6
    assert H.hif8_pts_search(16, 16, H.BF16, 0, 16, N, M, N, K, -4, 5, 16, 16, 256, 8, check=False) == 8
