"""Batch-sharded (data-parallel) gradient quantization and weight gradient: argument marshalling
around the staged entry points of the library, with the exchanges between them.

Every rank holds `N_local` images of the layer's tensors.  The statistics, density counts, classes and
clip values of Algorithm 1 belong to the whole batch; the stages compute the local parts on the GPU
and `Collective` exchanges the per-channel scalars (broadcast of the pivot, maximum of |g|max, sum of
the moments, sum of the counts, integer sum of the weight-gradient accumulators).  No arithmetic of the
method happens here.

`Collective` wraps `torch.distributed` (NCCL on GPUs, gloo on CPU); the tests also drive the same
stage functions with an in-process collective over several shards on one GPU, one stage at a time for
all shards, which is how more ranks than GPUs are emulated.
"""
from dataclasses import dataclass
from typing import List, Optional


class Collective:
    """The exchanges the sharded step needs, over a torch.distributed process group."""

    def __init__(self, dist, group=None):
        self.dist, self.group = dist, group

    def broadcast(self, t, src=0):
        self.dist.broadcast(t, src=src, group=self.group)

    def all_max(self, t):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)

    def all_sum(self, t):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)


@dataclass
class GradShard:
    """One rank's operands of the gradient quantizer (device tensors; dY is NHWC)."""
    dY: object
    N_local: int
    first_image: int
    vq: object
    gq: Optional[object]
    s_state: object
    cls: Optional[object]
    gmax_layer: object
    ws: object
    # scratch of the stages, [C] each (sums: [2][C] float64, cnt: int64)
    pivot: object = None
    absmax: object = None
    sums: object = None
    mean: object = None
    sigma: object = None
    cnt: object = None


def alloc_stage_buffers(sh: GradShard, C: int, torch) -> None:
    dev = sh.dY.device
    f32 = dict(dtype=torch.float32, device=dev)
    sh.pivot, sh.absmax = torch.zeros(C, **f32), torch.zeros(C, **f32)
    sh.mean, sh.sigma = torch.zeros(C, **f32), torch.zeros(C, **f32)
    sh.sums = torch.zeros(2 * C, dtype=torch.float64, device=dev)
    sh.cnt = torch.zeros(C, dtype=torch.int64, device=dev)


# Stage functions: `kernels` is the binding module (paper_2102_04782_b200.api).  Between two stages the
# caller runs the exchange named in the comment on the listed tensors.
def stage_pivot(kernels, sh: GradShard, C: int) -> None:
    """pivot = the channel values of the shard's first pixel; exchange afterwards: broadcast from the first rank."""
    kernels.dp_grad_pivot(sh.dY, kernels.NHWC, C, sh.pivot)


def stage_moments(kernels, sh: GradShard, C, H, W) -> None:
    """exchange afterwards: all_max(absmax), all_sum(sums)."""
    kernels.dp_grad_moments(sh.dY, kernels.NHWC, sh.N_local, C, H, W, sh.pivot, sh.absmax, sh.sums, sh.ws)


def stage_sigma_count(kernels, sh: GradShard, C, H, W, M_global, params) -> None:
    """exchange afterwards: all_sum(cnt)."""
    kernels.dp_grad_sigma(sh.absmax, sh.sums, sh.pivot, C, M_global, params, sh.mean, sh.sigma, sh.gmax_layer)
    kernels.dp_grad_count(sh.dY, kernels.NHWC, sh.N_local, C, H, W, sh.sigma, sh.cnt, sh.ws)


def stage_solve_codes(kernels, sh: GradShard, C, H, W, M_global, params, has_prev, seed) -> None:
    kernels.dp_grad_solve(sh.cnt, sh.absmax, C, M_global, params, sh.s_state, has_prev, sh.cls)
    kernels.dp_grad_codes(sh.dY, kernels.NHWC, sh.N_local, C, H, W, sh.first_image, sh.s_state, sh.gmax_layer, seed,
                          sh.vq, sh.gq)


def quantize_grad_sharded(kernels, coll: Collective, sh: GradShard, C: int, H: int, W: int, N_global: int,
                          params, has_prev: bool, seed: int) -> None:
    """Algorithm 1's gradient quantization on this rank's shard of a batch of N_global images."""
    M = N_global * H * W
    stage_pivot(kernels, sh, C)
    coll.broadcast(sh.pivot, src=0)
    stage_moments(kernels, sh, C, H, W)
    coll.all_max(sh.absmax)
    coll.all_sum(sh.sums)
    stage_sigma_count(kernels, sh, C, H, W, M, params)
    coll.all_sum(sh.cnt)
    stage_solve_codes(kernels, sh, C, H, W, M, params, has_prev, seed)


def conv_bwd_filter_sharded(kernels, coll: Collective, qX, vq, sX, s_state, geom, acc_i32, dW, ws) -> None:
    """dW of the whole batch from this rank's codes: integer partial, exact integer sum over the ranks
    (all ranks quantized with the same scales), then Eq. 7."""
    kernels.conv_bwd_filter(qX, vq, sX, s_state, geom, acc_i32, ws)
    coll.all_sum(acc_i32)
    per_cout = acc_i32.numel() // geom.Cout
    kernels.dequant_filter(acc_i32, sX, s_state, geom.Cout, per_cout, dW)


def quantize_activation_sharded(kernels, coll: Collective, x, layout, N_local, C, H, W, sX, qX, ws=None) -> None:
    """Layer-wide codes of X with the scale of the whole batch: local max, maximum over ranks, codes."""
    kernels.absmax(x, sX)
    coll.all_max(sX)
    kernels.quantize_tensor(x, layout, N_local, C, H, W, kernels.SCALE_GIVEN, sX, kernels.ROUND_NEAREST_EVEN, 0, qX, ws)


class LockstepCollective:
    """Several shards in one process (one GPU): the exchange acts on the list of all shards' tensors.
    Used by driving the stage functions for every shard, then calling these on the lists."""

    @staticmethod
    def broadcast(tensors: List, src=0):
        for i, t in enumerate(tensors):
            if i != src:
                t.copy_(tensors[src])

    @staticmethod
    def all_max(tensors: List):
        m = tensors[0].clone()
        for t in tensors[1:]:
            m = m.maximum(t)
        for t in tensors:
            t.copy_(m)

    @staticmethod
    def all_sum(tensors: List):
        s = tensors[0].clone()
        for t in tensors[1:]:
            s = s + t              # rank order, as a ring all-reduce of a fixed world size would fix it
        for t in tensors:
            t.copy_(s)
