"""Tensor-parallel sharding and exchange on CPU: the shards partition the stored weight without
touching a group (column shards concatenate to the unsharded outputs, row shards sum to them), bad
splits are refused, and a world-size-2 gloo run of the MLP block returns the sum of the ranks'
partial outputs on every rank."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2505_14638_b200 import inputs, tp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _weights(N, K, seed, asym=False):
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, seed), symmetric=not asym,
                                                           per_channel=asym)
    return tp.Weights(codes, gscale, gzero, s_w)


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("asym", [False, True])
def test_column_shards_are_the_unsharded_output_channels(world, asym):
    N, K, M = 256, 512, 5
    w = _weights(N, K, 3, asym)
    x8, s_x = oracle.quantize_act(inputs.make_activation(M, K, 4))
    full = oracle.linear(x8, s_x, oracle.dequant_weight(w.codes, w.gscale, w.gzero), w.s_w, want=("y64",))["y64"]
    per = N // world
    for r in range(world):
        s = tp.column_shard(w, r, world)
        assert s.N == per and s.K == K
        got = oracle.linear(x8, s_x, oracle.dequant_weight(s.codes, s.gscale, s.gzero), s.s_w, want=("y64",))["y64"]
        assert np.array_equal(got, full[:, r * per:(r + 1) * per])


def test_stacked_column_shard_takes_the_same_slice_of_gate_and_up():
    F, K, world = 192, 256, 3
    w = _weights(2 * F, K, 5, asym=True)
    per = F // world
    for r in range(world):
        s = tp.column_shard(w, r, world, stacked=2)
        rows = np.r_[r * per:(r + 1) * per, F + r * per:F + (r + 1) * per]
        assert np.array_equal(s.codes, w.codes[rows]) and np.array_equal(s.gscale, w.gscale[rows])
        assert np.array_equal(s.gzero, w.gzero[rows]) and np.array_equal(s.s_w, w.s_w[rows])
        assert s.codes.flags["C_CONTIGUOUS"]


@pytest.mark.parametrize("world", [1, 2, 4])
def test_row_shards_keep_groups_whole_and_sum_to_the_unsharded_product(world):
    N, K, M = 64, 1024, 3
    w = _weights(N, K, 7, asym=True)
    w8 = oracle.dequant_weight(w.codes, w.gscale, w.gzero)
    x8, s_x = oracle.quantize_act(inputs.make_activation(M, K, 8))
    full = oracle.linear(x8, s_x, w8, w.s_w, want=("y64",))["y64"]
    per = K // world
    total = np.zeros_like(full)
    for r in range(world):
        s = tp.row_shard(w, r, world)
        assert s.K == per and s.gscale.shape == (N, per // 128) and s.s_w is w.s_w
        w8_r = oracle.dequant_weight(s.codes, s.gscale, s.gzero)
        assert np.array_equal(w8_r, w8[:, r * per:(r + 1) * per])            # every group with its own scale
        x8_r = np.ascontiguousarray(tp.row_shard_input(x8, r, world))
        total += oracle.linear(x8_r, s_x, w8_r, w.s_w, want=("y64",))["y64"]
    assert np.allclose(total, full, rtol=1e-12, atol=1e-300)


def test_splits_that_would_cut_a_group_or_misalign_the_kernel_are_refused():
    w = _weights(96, 384, 9)
    with pytest.raises(ValueError):
        tp.row_shard(w, 0, 2)            # 192 columns per rank: one and a half groups
    with pytest.raises(ValueError):
        tp.column_shard(w, 0, 4)         # 24 channels per rank: not a multiple of 16
    with pytest.raises(ValueError):
        tp.column_shard(w, 2, 2)
    with pytest.raises(ValueError):
        tp.column_shard(w, 0, 1, stacked=5)
    tp.row_shard(w, 2, 3)
    tp.column_shard(w, 1, 2)
    tp.column_shard(w, 0, 3, stacked=2)  # 48 per block, 16 per rank
    with pytest.raises(ValueError):
        tp.TPMlpBlock(_weights(64, 128, 1), _weights(128, 64, 2), 0, 1, ops=object())   # gate/up is not 2 F x H


WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"]); sys.path.insert(0, os.path.join(os.environ["REPO_ROOT"], "tests"))
import numpy as np, torch, torch.distributed as dist
import oracle
from paper_2505_14638_b200 import inputs, tp
from tp_ops import OracleOps, bf16_tensor_bits
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
H, F, M = 256, 512, 6
def weights(N, K, seed):
    return tp.Weights(*oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.05, seed), symmetric=True))
gu, down = weights(2 * F, H, 11), weights(H, F, 12)
x = inputs.make_activation(M, H, 13)
ops = OracleOps()
for fp32 in (True, False):
    blk = tp.TPMlpBlock(gu, down, rank, world, ops=ops, exchange=tp.Exchange(), reduce_fp32=fp32)
    y = blk.forward(x)
    # every rank recomputes all partial outputs serially and sums them itself
    parts = [tp.TPMlpBlock(gu, down, r, world, ops=ops, exchange=tp.Exchange(world=world), reduce_fp32=fp32).partial(x)
             for r in range(world)]
    want = parts[0].clone()
    for p in parts[1:]:
        want += p
    assert y.dtype == (torch.float32 if fp32 else torch.bfloat16)
    assert torch.equal(y, want), (rank, fp32)
    # and the sharded block stays close to the unsharded one (same weights; the down projection's
    # activations are quantized per rank slice instead of per whole row)
    one = tp.TPMlpBlock(gu, down, 0, 1, ops=ops, exchange=tp.Exchange(world=1), reduce_fp32=True).forward(x)
    err = (y.float() - one).norm() / one.norm()
    assert err < 0.03, float(err)
    gathered = [torch.empty_like(y) for _ in range(world)]
    dist.all_gather(gathered, y)
    assert all(torch.equal(g, y) for g in gathered)                       # replicated result
dist.barrier()
if rank == 0:
    print("OK", world, flush=True)
dist.destroy_process_group()
"""


def test_mlp_block_world_size_2_gloo(tmp_path):
    script = tmp_path / "tp_worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29741", str(script)]
    res = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-3000:]
    assert "OK 2" in res.stdout
