"""Per-tensor scaled conversion of a tensor that is sharded over the ranks of a process group.

Section 5.1 defines one scale factor per GEMM input tensor; when the tensor lives as one shard per GPU, the amax
behind that factor is the maximum over all shards.  The data path is three steps, none of which returns to the host:

    hif8_amax(shard)                      -> 4-byte device value per rank
    all_reduce(MAX) over the group        -> the tensor's amax on every rank (NCCL over NVLink; latency only)
    hif8_encode_from_amax(shard, amax)    -> each rank converts its shard with the common exponent

The GEMM shards the same way the paper's layers do: the weight bytes are split along N (`shard_range` gives each rank a
block of whole 256-column tiles), every rank multiplies the full activation by its block and owns that block of C --
no collective on the data path (`column_sharded_gemm`).

This module is marshalling around those calls; `ops` is the binding module (injected so that the host logic can be
exercised without a GPU).  torch.distributed is the plumbing: NCCL for CUDA tensors, gloo in the CPU tests.
"""
import torch
import torch.distributed as dist


def sharded_amax_scale_encode(ops, shard, src_dtype, dst, n, target_exp, rnd, flags, seed, d_amax, workspace, workspace_bytes,
                              d_scale_exp_out=None, group=None, stream=None):
    """Convert this rank's `shard` (n elements) with the scale exponent of the whole tensor.

    d_amax: one float32 element on the shard's device; on return it holds the amax of the whole tensor.
    With no initialised process group (or a group of one) this is hif8_amax + hif8_encode_from_amax."""
    ops.hif8_amax(shard, src_dtype, n, d_amax, workspace, workspace_bytes, stream)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        if stream is not None and d_amax.is_cuda:
            with torch.cuda.stream(stream):
                dist.all_reduce(d_amax, op=dist.ReduceOp.MAX, group=group)
        else:
            dist.all_reduce(d_amax, op=dist.ReduceOp.MAX, group=group)
    ops.hif8_encode_from_amax(shard, src_dtype, dst, n, target_exp, rnd, flags, seed, d_amax, d_scale_exp_out, None, stream)
    return d_amax


def shard_range(n, world, rank, align=1):
    """[lo, hi) of rank `rank` when n units are dealt out in `world` contiguous pieces whose boundaries are multiples of
    `align` (the last piece takes the ragged end).  Pieces differ by at most `align` units and tile [0, n) exactly."""
    units = -(-n // align)
    lo = (units * rank // world) * align
    hi = (units * (rank + 1) // world) * align
    return min(lo, n), min(hi, n)


def column_sharded_gemm(ops, Aq, Wq_shard, C_shard, M, n_local, K, d_scale_exp_a, d_scale_exp_w, workspace, workspace_bytes,
                        c_dtype=None, stream=None):
    """This rank's column block of C = dec(Aq) dec(Wq) * 2^-(sa+sw): Wq_shard is [K, n_local] (contiguous), C_shard
    [M, n_local].  The per-tensor exponents are those of the whole tensors, so the blocks of all ranks put side by side
    are the product of the unsharded call."""
    if n_local == 0:
        return
    ops.hif8_gemm(Aq, K, Wq_shard, n_local, 0, C_shard, n_local, ops.BF16 if c_dtype is None else c_dtype, M, n_local, K,
                  d_scale_exp_a, d_scale_exp_w, workspace, workspace_bytes, stream)
