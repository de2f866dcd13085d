"""Tensor-parallel W4A8 linear layers and the MLP block built from them (the multi-device
deployment behind the paper's end-to-end comparison, Sec. 4.3 / Fig. 4: one decoder block whose
weights are split over the devices of a node).

Sharding keeps the stored format (Sec. 3.2, Eq. 6-9: INT4 codes, one BF16 scale per group of 128
consecutive input columns, an FP8-range scale s_w per output channel or per tensor) intact:

* column-parallel: output channels (rows of the stored [N, K] weight) are split; every rank holds
  whole rows with all their groups, takes the replicated activations and produces its slice of the
  outputs -- no exchange;
* row-parallel: input columns are split at group boundaries (multiples of 128), so every group and
  its scale stay on one rank; every rank multiplies its slice of the activations (quantized per
  token over that slice, Eq. 13) with its slice of the weights, and the partial outputs are summed
  over the ranks -- the one exchange step of the block (an all-reduce).

A gated MLP block is column-parallel (stacked gate/up projection) followed by row-parallel (down
projection): the activation between them never leaves the rank.  The attention projections of a
decoder block use the same two classes (qkv column-parallel, o row-parallel).

The arithmetic runs in the CUDA library through `CudaOps`; nothing here computes.  `ops` can be
replaced by any object with the same four methods (the tests drive the sharding and the exchange
on CPU that way).
"""
from dataclasses import dataclass

GROUP = 128
N_ALIGN = 16      # the linear kernels want a multiple of 16 output channels


@dataclass
class Weights:
    """Canonical stored weight of one linear layer: codes u8 [N, K/2] (two codes per byte), gscale
    BF16 bits [N, K/128], gzero u8 [N, K/128] or None (zero-point 8), s_w float32 [N] or [1]."""
    codes: object
    gscale: object
    gzero: object
    s_w: object

    @property
    def N(self):
        return self.codes.shape[0]

    @property
    def K(self):
        return self.codes.shape[1] * 2


def _even_split(total, world, unit, what):
    if world < 1 or total % world != 0 or (total // world) % unit != 0:
        raise ValueError("%s = %d does not split over %d ranks in multiples of %d" % (what, total, world, unit))
    return total // world


def column_shard(w: Weights, rank: int, world: int, stacked: int = 1) -> Weights:
    """Rows (output channels) of `w` owned by `rank`.  `stacked` = number of equal blocks stacked
    along N (2 for a gate/up projection stored as [gate; up]): the rank takes the same slice of
    every block, stacked in the same order, so its output is [gate slice, up slice]."""
    if not 0 <= rank < world:
        raise ValueError("rank %d outside world of %d" % (rank, world))
    if stacked < 1 or w.N % stacked != 0:
        raise ValueError("N = %d is not %d stacked blocks" % (w.N, stacked))
    block = w.N // stacked
    per = _even_split(block, world, N_ALIGN, "output channels per block")
    rows = [slice(b * block + rank * per, b * block + (rank + 1) * per) for b in range(stacked)]

    def take(a):
        if a is None:
            return None
        parts = [a[r] for r in rows]
        return parts[0] if len(parts) == 1 else _cat(parts)

    s_w = w.s_w if _numel(w.s_w) == 1 else take(w.s_w)
    return Weights(take(w.codes), take(w.gscale), take(w.gzero), s_w)


def row_shard(w: Weights, rank: int, world: int) -> Weights:
    """Input columns of `w` owned by `rank`, cut at group boundaries: K/world columns, i.e.
    K/(2 world) code bytes and K/(128 world) groups per row; s_w is shared by all ranks."""
    if not 0 <= rank < world:
        raise ValueError("rank %d outside world of %d" % (rank, world))
    per = _even_split(w.K, world, GROUP, "input columns")
    k0, k1 = rank * per, (rank + 1) * per
    cut = lambda a, d: None if a is None else _contig(a[:, k0 // d:k1 // d])
    return Weights(cut(w.codes, 2), cut(w.gscale, GROUP), cut(w.gzero, GROUP), w.s_w)


def row_shard_input(x, rank: int, world: int):
    """The slice of replicated activations [M, K] that goes with row_shard(w, rank, world)."""
    per = _even_split(x.shape[1], world, GROUP, "input columns")
    return x[:, rank * per:(rank + 1) * per]


def _numel(a):
    return a.numel() if hasattr(a, "numel") else a.size


def _cat(parts):
    if hasattr(parts[0], "numel"):
        import torch
        return torch.cat(parts, dim=0).contiguous()
    import numpy as np
    return np.ascontiguousarray(np.concatenate(parts, axis=0))


def _contig(a):
    if hasattr(a, "contiguous"):
        return a.contiguous()
    import numpy as np
    return np.ascontiguousarray(a)


class CudaOps:
    """The four steps of the block on the CUDA library (raises when it is missing)."""

    def __init__(self):
        from . import binding
        binding.lib()
        self.b = binding

    def prepare(self, w: Weights):
        return self.b.prepack_weight(w.codes, w.gscale, w.gzero, w.s_w)

    def quantize_act(self, x):
        return self.b.quantize_act(x)

    def linear(self, x8, s_x, prepared, fp32_out):
        # one workspace per (layer, token count), kept with the layer: zero-filled when created and
        # left clean by every launch
        cache = prepared.__dict__.setdefault("_tp_workspaces", {})
        ws = cache.get(x8.shape[0])
        if ws is None:
            ws = self.b.new_workspace(x8.shape[0], prepared.N, prepared.K, prepared.fmt, x8.device)
            cache[x8.shape[0]] = ws
        return self.b.linear_tiled(x8, s_x, prepared, out_dtype=self.b.OUT_FP32 if fp32_out else self.b.OUT_BF16,
                                   workspace=ws)

    def silu_mul_quantize(self, gate_up):
        return self.b.silu_mul_quantize(gate_up)


class Exchange:
    """Sum over the ranks of a process group (torch.distributed; NCCL on GPUs, gloo on CPU)."""

    def __init__(self, group=None, world=None):
        self.group = group
        if world is None:
            import torch.distributed as dist
            world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.world = world

    def all_reduce_sum(self, y):
        if self.world > 1:
            import torch.distributed as dist
            dist.all_reduce(y, op=dist.ReduceOp.SUM, group=self.group)
        return y


class ColumnParallelLinear:
    """This rank's output channels of a W4A8 linear layer; inputs replicated, no exchange."""

    def __init__(self, w: Weights, rank, world, stacked=1, ops=None):
        self.ops = ops if ops is not None else CudaOps()
        self.shard = column_shard(w, rank, world, stacked)
        self.prepared = self.ops.prepare(self.shard)

    def forward_quantized(self, x8, s_x, fp32_out=False):
        return self.ops.linear(x8, s_x, self.prepared, fp32_out)

    def forward(self, x, fp32_out=False):
        x8, s_x = self.ops.quantize_act(x)
        return self.forward_quantized(x8, s_x, fp32_out)


class RowParallelLinear:
    """This rank's input columns of a W4A8 linear layer.  The input is this rank's slice of the
    activations (already quantized, or BF16 to be quantized per token over the slice); the partial
    outputs are summed over the ranks.  `reduce_fp32`: exchange FP32 partial sums (the result is
    FP32) instead of BF16 ones."""

    def __init__(self, w: Weights, rank, world, ops=None, exchange=None, reduce_fp32=False):
        self.ops = ops if ops is not None else CudaOps()
        self.exchange = exchange if exchange is not None else Exchange(world=world)
        if self.exchange.world != world:
            raise ValueError("exchange spans %d ranks, the shard plan %d" % (self.exchange.world, world))
        self.shard = row_shard(w, rank, world)
        self.prepared = self.ops.prepare(self.shard)
        self.reduce_fp32 = reduce_fp32

    def partial_quantized(self, x8, s_x):
        return self.ops.linear(x8, s_x, self.prepared, self.reduce_fp32)

    def forward_quantized(self, x8, s_x):
        return self.exchange.all_reduce_sum(self.partial_quantized(x8, s_x))

    def forward(self, x_slice):
        x8, s_x = self.ops.quantize_act(x_slice)
        return self.forward_quantized(x8, s_x)


class TPMlpBlock:
    """Gated MLP block over `world` ranks: quantize(x) -> gate/up (column-parallel, stacked
    [gate; up]) -> silu(gate) * up fused with the quantization of the down projection's input ->
    down (row-parallel) -> all-reduce.  x is replicated; the result is replicated."""

    def __init__(self, gate_up: Weights, down: Weights, rank, world, ops=None, exchange=None, reduce_fp32=False):
        if gate_up.N % 2 != 0 or gate_up.N // 2 != down.K or gate_up.K != down.N:
            raise ValueError("gate/up [%d, %d] and down [%d, %d] do not form an MLP block"
                             % (gate_up.N, gate_up.K, down.N, down.K))
        ops = ops if ops is not None else CudaOps()
        self.ops = ops
        self.gate_up = ColumnParallelLinear(gate_up, rank, world, stacked=2, ops=ops)
        self.down = RowParallelLinear(down, rank, world, ops=ops, exchange=exchange, reduce_fp32=reduce_fp32)

    def partial(self, x):
        """This rank's partial output, before the exchange."""
        gu = self.gate_up.forward(x)
        h8, s_h = self.ops.silu_mul_quantize(gu)
        return self.down.partial_quantized(h8, s_h)

    def forward(self, x):
        return self.down.exchange.all_reduce_sum(self.partial(x))
