"""The sharded per-tensor scaling path under a real process group on CPU (gloo, world size 2): every rank must end up
with the amax and the scale exponent of the WHOLE tensor, and its codes must be the corresponding slice of the
oracle's conversion of the whole tensor.  The device calls are replaced by a stand-in with the same names that
computes on numpy through the oracle (test infrastructure), so only the collective logic of sharded.py is under test
here; the CUDA entry points behind those names are covered by tests/test_gpu_sharded.py."""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


class OracleOps:
    """hif8_amax / hif8_encode_from_amax on CPU tensors, through the oracle."""

    def __init__(self):
        from oracle import hif8_oracle as O
        self.O = O

    def hif8_amax(self, src, dtype, n, d_amax, ws, wsb, stream=None):
        d_amax[0] = self.O.amax_scale(src.numpy()[:n], dtype, 14)[0]

    def hif8_encode_from_amax(self, src, dtype, dst, n, target, rnd, flags, seed, d_amax, d_se_out=None, d_scale_out=None,
                              stream=None):
        a = float(d_amax[0])
        se = 0 if a == 0 else int(np.clip(target - int(np.floor(np.log2(a))), -126, 126))
        dst[:n] = torch.from_numpy(self.O.encode(src.numpy()[:n], dtype, se, rnd, flags, seed, quick=True))
        if d_se_out is not None:
            d_se_out[0] = se


def _full_tensor():
    import workloads as W
    x = W.normal_f32(2 * 5000, 77)
    x[7000] = 300.0        # the maximum lives in rank 1's shard
    x[100] = np.inf        # non-finite values do not count
    return x


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2409_16626_b200 import sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = _full_tensor()
    n = x.size // world
    shard = torch.from_numpy(x[rank * n:(rank + 1) * n].copy())
    dst = torch.zeros(n, dtype=torch.uint8)
    d_amax = torch.zeros(1, dtype=torch.float32)
    d_se = torch.zeros(1, dtype=torch.int32)
    sharded.sharded_amax_scale_encode(OracleOps(), shard, 0, dst, n, 14, 0, 0, 0, d_amax, None, 0, d_se)
    json.dump({"amax": float(d_amax[0]), "se": int(d_se[0]), "codes": dst.numpy().tolist()}, open(f"{out}.{rank}", "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_scaling_uses_the_amax_of_the_whole_tensor_gloo(tmp_path):
    from oracle import hif8_oracle as O
    out = str(tmp_path / "r")
    mp.spawn(_worker, args=(2, 31000 + os.getpid() % 2000, out), nprocs=2, join=True)
    x = _full_tensor()
    amax, se = O.amax_scale(x, O.F32, 14)
    ref = O.encode(x, O.F32, se, O.TA)
    assert amax == 300.0
    for rank in range(2):
        r = json.load(open(f"{out}.{rank}"))
        assert r["amax"] == amax and r["se"] == se
        assert np.array_equal(np.array(r["codes"], dtype=np.uint8), ref[rank * 5000:(rank + 1) * 5000])
    # a rank scaling by its own shard alone would have used another exponent
    assert O.amax_scale(x[:5000], O.F32, 14)[1] != se


def test_without_a_process_group_it_is_the_two_local_calls():
    from paper_2409_16626_b200 import sharded
    from oracle import hif8_oracle as O
    x = _full_tensor()
    dst = torch.zeros(x.size, dtype=torch.uint8)
    d_amax = torch.zeros(1)
    sharded.sharded_amax_scale_encode(OracleOps(), torch.from_numpy(x.copy()), 0, dst, x.size, 14, 0, 0, 0, d_amax, None, 0)
    amax, se = O.amax_scale(x, O.F32, 14)
    assert float(d_amax[0]) == amax and np.array_equal(dst.numpy(), O.encode(x, O.F32, se, O.TA))


# ------------------------------------------------------------------------------------------------------------
# GEMM sharded along N: every rank owns whole 256-column tiles of Wq and of C; no collective on the data path
# ------------------------------------------------------------------------------------------------------------
class OracleGemmOps:
    """hif8_gemm on CPU tensors through the FP64 oracle (FP32 result), recording the shape each rank was handed."""
    BF16, F32 = 1, 0

    def __init__(self):
        from oracle import hif8_oracle as O
        self.O = O

    def hif8_gemm(self, Aq, lda, Wq, ldw, w_is_nk, C, ldc, c_dtype, M, N, K, d_sa, d_sw, ws, wsb, stream=None):
        assert lda == K and ldw == N and ldc == N and not w_is_nk
        sa, sw = int(d_sa[0]), int(d_sw[0])
        cs, _ = self.O.gemm_full(Aq.numpy().reshape(M, K), Wq.numpy().reshape(K, N), False, sa, sw)
        C.copy_(torch.from_numpy(cs.astype(np.float32)))


def _gemm_operands():
    import workloads as W
    return W.random_codes((40, 64), seed=5), W.random_codes((64, 1300), seed=6)   # N = 1300: five tiles and a ragged one


def _gemm_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2409_16626_b200 import sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    Aq, Wq = _gemm_operands()
    M, K = Aq.shape
    N = Wq.shape[1]
    c0, c1 = sharded.shard_range(N, world, rank, 256)
    w_shard = torch.from_numpy(np.ascontiguousarray(Wq[:, c0:c1]))
    C = torch.zeros(M, c1 - c0, dtype=torch.float32)
    sa, sw = torch.tensor([3], dtype=torch.int32), torch.tensor([-2], dtype=torch.int32)
    sharded.column_sharded_gemm(OracleGemmOps(), torch.from_numpy(Aq), w_shard, C, M, c1 - c0, K, sa, sw, None, 0, c_dtype=0)
    # the blocks are gathered only to check them; the method itself leaves C sharded by column
    blocks = [None] * world
    dist.all_gather_object(blocks, (c0, c1, C.numpy().tolist()))
    if rank == 0:
        json.dump(blocks, open(out, "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_column_sharded_gemm_blocks_tile_the_unsharded_product_gloo(tmp_path):
    from oracle import hif8_oracle as O
    out = str(tmp_path / "g.json")
    mp.spawn(_gemm_worker, args=(2, 33000 + os.getpid() % 2000, out), nprocs=2, join=True)
    Aq, Wq = _gemm_operands()
    full, _ = O.gemm_full(Aq, Wq, False, 3, -2)
    blocks = json.load(open(out))
    assert blocks[0][0] == 0 and blocks[-1][1] == Wq.shape[1] and blocks[0][1] == blocks[1][0]   # contiguous cover
    assert blocks[0][1] % 256 == 0                                                             # cut on a tile boundary
    got = np.concatenate([np.array(b[2], dtype=np.float32) for b in blocks], axis=1)
    assert np.array_equal(got, full.astype(np.float32))


def test_shard_range_tiles_exactly_for_any_world_size():
    from paper_2409_16626_b200 import sharded
    for n, align in ((28672, 256), (1300, 256), (16777216, 16), (5, 16), (0, 4), (1000003, 1)):
        for world in (1, 2, 3, 4, 8):
            prev = 0
            sizes = []
            for r in range(world):
                lo, hi = sharded.shard_range(n, world, r, align)
                assert lo == prev and lo <= hi <= n and (lo % align == 0 or lo == n)
                sizes.append(hi - lo)
                prev = hi
            assert prev == n
            assert max(sizes) - min(sizes) <= align or n < align * world
