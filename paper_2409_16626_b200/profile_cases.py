"""Run one named workload a few times, for use under a profiler:

    python -m paper_2409_16626_b200.profile_cases <case> [repeats]

cases: convert_f32 (FP32 4096^2: per-tensor scaled encode + decode), fq_bf16 (BF16 4096x8192 fake-quant, TA, HR and TE,
fused amax and given scale), encode_modes_f32 / encode_modes_bf16 (2^25 log-uniform values, every rounding mode), gemm (HiF8 GEMM
4096 x 7168 x 4096, fused and decode-once paths), gemm_forms (same size, decode-once path, the four operand layouts:
forward, dgrad form, wgrad form with FP32 accumulation, both transposed), gemm_narrow (16 x 8192 x 8192, the
weight-streaming kernel, weights as [K,N] and as [N,K]), channel_bf16 (per-channel scaled encode of a
BF16 8192 x 14336 weight, channel = column and channel = row, plus the overflow check of the same tensor), transpose_bf16
(BF16 8192 x 8192 to HiF8 bytes, flat and with transposed store, round half away and hybrid rounding).  Inputs are seeded device-side random tensors.
"""
import sys

import torch

from . import binding as H


def main():
    case = sys.argv[1] if len(sys.argv) > 1 else "convert_f32"
    reps = int(sys.argv[2]) if len(sys.argv) > 2 else 3
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    if case == "convert_f32":
        n = 4096 * 4096
        xs = [torch.randn(n, generator=g, device="cuda") for _ in range(3)]
        codes = torch.empty(n, dtype=torch.uint8, device="cuda")
        back = torch.empty(n, dtype=torch.float32, device="cuda")
        se = torch.zeros(1, dtype=torch.int32, device="cuda")
        for r in range(reps):
            H.hif8_amax_scale_encode(xs[r % 3], H.F32, codes, n, 14, H.RND_TA, 0, 0, None, None, se, None, ws, 256)
            H.hif8_decode(codes, back, H.F32, n, 12)
    elif case == "fq_bf16":
        n = 4096 * 8192
        xs = [torch.randn(n, generator=g, device="cuda").to(torch.bfloat16) for _ in range(3)]
        y = torch.empty_like(xs[0])
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR, H.RND_TE):
                H.hif8_fake_quant(xs[r % 3], y, H.BF16, n, 1, 14, mode, 0, 7, None, None, ws, 256)
                H.hif8_fake_quant(xs[r % 3], y, H.BF16, n, 0, 12, mode, 0, 7)
    elif case == "encode_modes_f32":
        n = 1 << 25
        e = torch.randint(-40, 20, (n,), generator=g, device="cuda", dtype=torch.int32) + 127
        m = torch.randint(0, 1 << 23, (n,), generator=g, device="cuda", dtype=torch.int32)
        bits = (e << 23) | m
        codes = torch.empty(n, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR):
                H.hif8_encode(bits, H.F32, codes, n, 0, mode, 0, 5)
    elif case == "encode_modes_bf16":
        n = 1 << 25
        e = torch.randint(-40, 20, (n,), generator=g, device="cuda", dtype=torch.int32) + 127
        m = torch.randint(0, 1 << 7, (n,), generator=g, device="cuda", dtype=torch.int32)
        bits = ((e << 7) | m).to(torch.int16)
        codes = torch.empty(n, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR, H.RND_SSR, H.RND_TE, H.RND_SR):
                H.hif8_encode(bits, H.BF16, codes, n, 0, mode, 0, 5)
    elif case == "transpose_bf16":
        R, C = 8192, 8192
        xs = [torch.randn(R * C, generator=g, device="cuda").to(torch.bfloat16) for _ in range(2)]
        codes = torch.empty(R * C, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            for mode in (H.RND_TA, H.RND_HR):
                H.hif8_encode(xs[r & 1], H.BF16, codes, R * C, 3, mode, 0, 5)
                H.hif8_encode_transpose(xs[r & 1], H.BF16, codes, R, C, 3, None, mode)
    elif case == "gemm":
        M, N, K = 4096, 7168, 4096
        A = torch.randint(0, 256, (M, K), dtype=torch.uint8, device="cuda", generator=g)
        W = torch.randint(0, 256, (K, N), dtype=torch.uint8, device="cuda", generator=g)
        for t in (A, W):                                   # keep the operands finite
            t[(t == 0x80) | ((t & 0x7F) == 0x6F)] = 0x08
        C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        big = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
        gws = torch.empty(big, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            H.hif8_gemm(A, K, W, N, 0, C, N, H.BF16, M, N, K, None, None, gws, big)
            H.hif8_gemm(A, K, W, N, 0, C, N, H.BF16, M, N, K, None, None, gws, 256)
    elif case == "gemm_narrow":
        M, N, K = 16, 8192, 8192
        A = torch.randint(8, 100, (M * K,), dtype=torch.uint8, device="cuda", generator=g)
        W = torch.randint(8, 100, (K * N,), dtype=torch.uint8, device="cuda", generator=g)
        C = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        for r in range(reps):
            H.hif8_gemm(A, K, W, N, 0, C, N, H.BF16, M, N, K, None, None, ws, 256)
            H.hif8_gemm(A, K, W, K, 1, C, N, H.BF16, M, N, K, None, None, ws, 256)
    elif case == "gemm_forms":
        M, N, K = 4096, 7168, 4096
        A = torch.randint(8, 100, (M * K,), dtype=torch.uint8, device="cuda", generator=g)
        W = torch.randint(8, 100, (K * N,), dtype=torch.uint8, device="cuda", generator=g)
        Cb = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
        Cf = torch.zeros(M, N, dtype=torch.float32, device="cuda")
        big = H.hif8_workspace_bytes(H.WS_GEMM, M * K + K * N)
        gws = torch.empty(big, dtype=torch.uint8, device="cuda")
        for r in range(reps):
            H.hif8_gemm_ex(A, K, 0, W, N, 0, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
            H.hif8_gemm_ex(A, K, 0, W, K, 1, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
            H.hif8_gemm_ex(A, M, 1, W, N, 0, Cf, N, H.F32, M, N, K, None, None, None, 1, gws, big)
            H.hif8_gemm_ex(A, M, 1, W, K, 1, Cb, N, H.BF16, M, N, K, None, None, None, 0, gws, big)
    elif case == "channel_bf16":
        K, N = 8192, 14336
        w = (torch.randn(K, N, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
        q = torch.empty(K * N, dtype=torch.uint8, device="cuda")
        amax = torch.empty(N, dtype=torch.float32, device="cuda")
        se = torch.empty(N, dtype=torch.int32, device="cuda")
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        for r in range(reps):
            H.hif8_channel_amax_scale_encode(w, H.BF16, q, K, N, 1, 14, H.RND_TA, 0, 0, None, amax, se)
            H.hif8_channel_amax_scale_encode(w, H.BF16, q, N, K, 0, 14, H.RND_TA, 0, 0, None, amax, se)
            H.hif8_check_finite(w, H.BF16, K * N, flag)
    else:
        raise SystemExit(f"unknown case {case}")
    torch.cuda.synchronize()
    print("done", case, H.hif8_launch_count())


if __name__ == "__main__":
    main()
