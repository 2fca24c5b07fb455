"""Token-sharded data parallelism of one melded layer: every rank holds a full replica of the layer (backbone with the
melded adapter rows, DeltaBuffer) and a shard of the tokens.  The method has exactly one exchange step per layer and
training step -- the sum of the adapter gradients dB over the shards (Alg. 3 line 3 is a contraction over the tokens) --
plus three scalar maxima, because the per-tensor FP8 scales of X, O_A and dY (Eq. quantize) are those of the whole
tensors, not of a shard: with the maxima combined first, every shard is cast with the scale the unsharded tensor would
get, so a shard's Y, O_A and dX are bit for bit the rows the unsharded call would produce.  After the exchange every rank
runs the identical, deterministic proxy update (Alg. 3 lines 4-6) on the summed gradient, so the replicas stay identical
without ever exchanging the backbone.

The class is split into phases so that it can be driven in two ways: `step()` runs all phases with collectives of a
communicator (by default `torch.distributed` on the default group: NCCL between GPUs, gloo between CPU ranks in the
tests); a test on a single device runs the phases of several replicas one after another and combines the values
itself.  `ops` is the module that provides the layer calls (by default the ctypes binding of the CUDA library; there is
no CPU implementation in this package).  Per-tensor scaled layers only.

The benchmark does not use this: its configurations are single-GPU, and `bench.py --gpus N` runs independent replicas."""
from __future__ import annotations

import torch


class DistComm:
    """In-place all-reduces over a torch.distributed process group."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group

    def all_reduce_max(self, t: torch.Tensor):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)

    def all_reduce_sum(self, t: torch.Tensor):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)


class SideStream:
    """Where the exchange of dB runs while the compute stream goes on with the input-gradient product.  On a CUDA device:
    a second stream and two events (fork: the side stream waits for what the compute stream has enqueued so far; join:
    the compute stream waits for what the side stream has enqueued).  Without one (CPU tensors, in the tests): both are
    no-ops and the calls simply run in program order."""

    def __init__(self, device=None):
        self.cuda = device is not None and torch.device(device).type == "cuda"
        if self.cuda:
            self.stream = torch.cuda.Stream(device=device)
            self.forked, self.joined = torch.cuda.Event(), torch.cuda.Event()

    def fork(self):
        if self.cuda:
            self.forked.record(torch.cuda.current_stream())
            self.stream.wait_event(self.forked)

    def run(self, fn):
        if self.cuda:
            with torch.cuda.stream(self.stream):
                fn()
        else:
            fn()

    def join(self):
        if self.cuda:
            self.joined.record(self.stream)
            torch.cuda.current_stream().wait_event(self.joined)


class TokenShardedLayer:
    def __init__(self, layer, ops=None, comm=None):
        if ops is None:
            from . import binding as ops      # fails loudly when the CUDA library is missing
        self.layer, self.ops, self.comm = layer, ops, comm
        self.side = None        # SideStream for the exchange of dB, created on first use
        self.OA = None          # this shard's O_A, saved by forward() for backward()
        self.amax_oa = None     # max |O_A|: of this shard after forward(), of all shards once combined

    # ---- phases ------------------------------------------------------------------------------------------------
    def input_absmax(self, X: torch.Tensor) -> torch.Tensor:
        """max |X| over this shard (fp32 [1]); combine with a MAX over the ranks before forward()."""
        return self.ops.absmax(X)

    def forward(self, X: torch.Tensor, amax_x: torch.Tensor, y_dtype=torch.bfloat16):
        """Y, O_A of this shard, cast with the scale of the whole X.  Leaves max |O_A| of this shard in self.amax_oa:
        combine it with a MAX over the ranks (in place) before backward()."""
        Y, self.OA, self.amax_oa, _ = self.ops.melded_forward(self.layer, X, y_dtype=y_dtype, amax_x=amax_x)
        return Y, self.OA

    def output_grad_absmax(self, dY: torch.Tensor) -> torch.Tensor:
        return self.ops.absmax(dY)

    def backward(self, dY: torch.Tensor, amax_dy: torch.Tensor, need_dx: bool = True, dx_dtype=torch.bfloat16):
        """dX of this shard and this shard's PARTIAL adapter gradient (fp32 [m, r]): sum it over the ranks before update()."""
        dX, dB, _ = self.ops.melded_backward(self.layer, dY, self.OA, self.amax_oa, need_dx=need_dx, dx_dtype=dx_dtype,
                                             amax_dy=amax_dy)
        return dX, dB

    def backward_db(self, dY: torch.Tensor, amax_dy: torch.Tensor):
        """The first half of backward(): the casts and this shard's partial dB.  Leaves the gradient codes behind for
        backward_dx()."""
        _, dB, _ = self.ops.melded_backward(self.layer, dY, self.OA, self.amax_oa, need_dx=False, amax_dy=amax_dy)
        return dB

    def backward_dx(self, T: int, dx_dtype=torch.bfloat16):
        """The second half: dX of this shard from the codes backward_db() left in the layer's workspace."""
        return self.ops.melded_backward_dx(self.layer, T, dx_dtype=dx_dtype)

    def update(self, dB_total: torch.Tensor, lr: float, k: int):
        """The proxy update with the summed gradient; identical on every rank."""
        return self.ops.proxy_update(self.layer, dB_total, lr, k)

    # ---- all phases, with collectives ------------------------------------------------------------------------------
    def step(self, X: torch.Tensor, dY: torch.Tensor, lr: float, k: int, y_dtype=torch.bfloat16, need_dx: bool = True,
             dx_dtype=torch.bfloat16, overlap: bool = True):
        comm = self.comm if self.comm is not None else DistComm()
        amax_x = self.input_absmax(X)
        comm.all_reduce_max(amax_x)
        Y, _ = self.forward(X, amax_x, y_dtype=y_dtype)
        comm.all_reduce_max(self.amax_oa)
        amax_dy = self.output_grad_absmax(dY)
        comm.all_reduce_max(amax_dy)
        if not (overlap and need_dx):
            dX, dB = self.backward(dY, amax_dy, need_dx=need_dx, dx_dtype=dx_dtype)
            comm.all_reduce_sum(dB)                   # the method's one exchange step: 4 m r bytes per layer
            return Y, dX, dB, self.update(dB, lr, k)
        # the exchange of dB overlaps the input-gradient product: nothing needs dB before the proxy update
        if self.side is None:
            self.side = SideStream(dY.device)
        dB = self.backward_db(dY, amax_dy)
        self.side.fork()                              # the side stream waits for dB ...
        self.side.run(lambda: comm.all_reduce_sum(dB))
        dX = self.backward_dx(dY.shape[0], dx_dtype=dx_dtype)   # ... while the compute stream goes on with dX
        self.side.join()                              # the update needs the summed dB
        idx = self.update(dB, lr, k)
        return Y, dX, dB, idx
