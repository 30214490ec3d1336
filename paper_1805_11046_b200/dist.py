"""Multi-GPU plumbing: one process per GPU over torch.distributed (NCCL on GPUs, gloo on CPU).

Two uses.  (1) Independent batches per rank (the benchmark's weak scaling): ranks share nothing on the data path;
the only exchanges are the max-over-ranks of a device time and the split of work units.  (2) One minibatch spread
over the ranks (data parallelism, Section 3: Range BN's mean and range are those of the whole minibatch): the path
then has four small exchange steps, all order-free reductions of a few numbers per channel or of integers --

    quantiser range of an activation / gradient tensor   (min, max)            MIN / MAX of 2 floats
    Range BN forward statistics per channel              (sum, min, max)       SUM fp64, MIN, MAX of C values
    Range BN backward sums per channel                   (sum dy, sum dy*xhat) SUM fp64 of 2C values
    weight gradient                                      int64 accumulators    SUM, exact

-- between calls of the library's split entry points (qbp_rangebn_fwd_stats / _apply, qbp_rangebn_bwd_stats /
_apply, qbp_bifurcate_shard, qbp_wgrad_s16 with acc_out, qbp_dequant_s64).  DataParallelLayer composes them.  The
reductions are plain torch.distributed all-reduces; a `reduce(tensor, op)` callable can stand in for them (the
single-GPU test runs the shards one after another and combines their partials itself).  No arithmetic of the
method happens here.
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment (torch.distributed.run)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def shard_units(total: int, rank: int, world: int):
    """[begin, end) of the `total` independent units (images, problems) that `rank` processes: contiguous,
    sizes differ by at most one, the union over ranks is exactly range(total)."""
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's time (all-reduce MAX); identity for a single process."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ------------------------------------------------------------------ exchange steps of a shared minibatch
def _all_reduce(t, op: str):
    """In-place all-reduce over the default process group; op in {"sum", "min", "max"}.  A no-op when
    torch.distributed is not initialised (one process)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return t
    dist.all_reduce(t, op={"sum": dist.ReduceOp.SUM, "min": dist.ReduceOp.MIN, "max": dist.ReduceOp.MAX}[op])
    return t


def allreduce_range(range_qp, reduce=_all_reduce):
    """range_qp: a qbp_qparams record [1, 4] (int32 storage) whose vmin / vmax are this rank's; afterwards they
    are the whole tensor's.  scale and zero_point are left alone (the quantiser derives them from the range)."""
    import torch
    f = range_qp.view(torch.float32)
    lo = f[:, 2].contiguous(); hi = f[:, 3].contiguous()
    reduce(lo, "min"); reduce(hi, "max")
    f[:, 2] = lo; f[:, 3] = hi
    return range_qp


def allreduce_bn_stats(col_sum, col_min, col_max, reduce=_all_reduce):
    """Per-channel (sum fp64, min, max) of this rank's rows -> of the whole minibatch."""
    reduce(col_sum, "sum"); reduce(col_min, "min"); reduce(col_max, "max")
    return col_sum, col_min, col_max


def allreduce_sums(*tensors, reduce=_all_reduce):
    for t in tensors:
        reduce(t, "sum")
    return tensors


class DataParallelLayer:
    """One quantised conv / linear layer + Range BN whose minibatch is spread over the ranks: every rank holds
    `rows` of the `rows_total` rows (batch x positions), starting at row `row_offset` of the whole minibatch.
    The calls are the library's own; between them sit the four exchange steps listed in the module docstring.
    With one rank (no reduce needed) the results are those of the undivided layer."""

    def __init__(self, B, conv=None, batch=0, in_features=0, out_features=0, relu=False, seed=0, tensor_id8=1,
                 tensor_id16=1, rows_total=None, row_offset=0, reduce=_all_reduce):
        self.B, self.conv, self.relu, self.reduce = B, conv, relu, reduce
        self.seed, self.id8, self.id16 = seed, tensor_id8, tensor_id16
        if conv is not None:
            self.rows, self.cin, self.cout = conv.N * conv.H * conv.W, conv.C, conv.K
        else:
            self.rows, self.cin, self.cout = batch, in_features, out_features
        self.rows_total = rows_total if rows_total is not None else self.rows
        self.row_offset = row_offset

    def forward(self, x, w, gamma=None, beta=None):
        import torch
        B = self.B
        self.gamma, self.beta = gamma, beta
        # quantiser range of the whole activation tensor, then this rank's codes under it
        xr = allreduce_range(B.qbp_range_chunked(x, 1), self.reduce)
        self.row_sums = torch.empty(self.rows, dtype=torch.int32, device=x.device) if self.conv is not None else None
        self.x_codes, self.qx = B.qbp_quantize_s8(x, range_in=xr, row_sums=self.row_sums)
        self.w_codes, self.qw = B.qbp_quantize_s8(w)                      # the weights are the same on every rank
        if self.conv is not None:
            _, self.z, _ = B.qbp_conv_s8_implicit(B.QBP_CONV_FPROP, self.conv, self.x_codes, self.qx, self.w_codes, self.qw)
        else:
            _, self.z, _ = B.qbp_gemm_s8(self.x_codes, self.qx, self.w_codes, self.qw)
        # Range BN over the whole minibatch: local statistics, exchange, apply
        stats = allreduce_bn_stats(*B.qbp_rangebn_fwd_stats(self.z), reduce=self.reduce)
        self.y, self.mean, self.vmin, self.vmax, _ = B.qbp_rangebn_fwd_apply(self.z, self.rows_total, *stats, gamma=gamma,
                                                                              beta=beta, relu=self.relu)
        return self.y

    def backward(self, dy):
        import torch
        B = self.B
        sums = B.qbp_rangebn_bwd_stats(dy, self.z, self.rows_total, self.mean, self.vmin, self.vmax, self.gamma, self.beta,
                                       self.relu)
        allreduce_sums(*sums, reduce=self.reduce)
        self.g, dgamma, dbeta = B.qbp_rangebn_bwd_apply(dy, self.z, self.rows_total, self.mean, self.vmin, self.vmax, *sums,
                                                        gamma=self.gamma, beta=self.beta, relu=self.relu)
        # both copies of the gradient under the whole tensor's range, each element with the random word of its
        # place in the whole tensor
        gr = allreduce_range(B.qbp_range_chunked(self.g, 1), self.reduce)
        rs8 = torch.empty(self.rows, dtype=torch.int32, device=dy.device) if self.conv is not None else None
        self.g8, self.qg8, self.ghi, self.glo, self.qg16 = B.qbp_bifurcate_shard(
            self.g, self.seed, self.id8, self.id16, self.row_offset * self.cout, gr, row_sums8=rs8)
        if self.conv is not None:
            _, dx, _ = B.qbp_conv_s8_implicit(B.QBP_CONV_DGRAD, self.conv, self.g8, self.qg8, self.w_codes, self.qw)
            acc, _, _ = B.qbp_wgrad_s16(self.x_codes, self.qx, self.ghi, self.glo, self.qg16, d=self.conv, want_acc=True, want_out=False)
        else:
            _, dx, _ = B.qbp_gemm_s8(self.g8, self.qg8, self.w_codes, self.qw, transB=True)
            acc, _, _ = B.qbp_wgrad_s16(self.x_codes, self.qx, self.ghi, self.glo, self.qg16, want_acc=True, want_out=False)
        # Eq. (grad_weight) over the whole minibatch: exact integer sum over the ranks, then one dequantisation
        self.reduce(acc, "sum")
        self.acc_dw = acc
        dw = B.qbp_dequant_s64(acc, self.qx, self.qg16)
        return dx, dw, dgamma, dbeta
