"""GPU: the decode-sized launches hand out their worker indices at run time (twice as many CTAs
as workers, at most one worker per SM and launch).  The state of a launch lives in the caller's
workspace, behind the split-K counters, and is cleared by the last CTA to enter; launches without
a workspace use an entry of a 64-entry table in the library image.  Whatever the placement, every
row range must be computed exactly once: long runs of launches -- more than the table has entries,
eager and replayed from one CUDA graph, alternating shapes, from two streams -- must reproduce the
first result bit for bit, and that result must match the oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_dev, weights_to_dev
from helpers import fp32_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed):
    W = inputs.make_weight(N, K, 0.02, seed)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    tw = binding.prepack_weight(*weights_to_dev(*wq), weight_format=binding.FMT_TILED_SIGNMAG)
    xb = inputs.make_activation(M, K, seed + 1)
    x8_ref, s_x_ref = oracle.quantize_act(xb)
    ref = oracle.linear(x8_ref, s_x_ref, oracle.dequant_weight(*wq[:3]), wq[3])
    x8, s_x = binding.quantize_act(bf16_dev(xb))
    ws = binding.new_workspace(M, N, K, tw.fmt, x8.device)
    return tw, x8, s_x, ref["y64"], ws


def test_many_launches_repeat_the_first_result():
    # K = 2048 and K = 4096 walk 16 and 32 k-blocks per tile (run-time worker indices);
    # N = 18960 gives ragged ranges, N = 37904 two tiles per worker
    cases = [_case(16, 18960, 2048, 5), _case(3, 37904, 4096, 7)]
    outs = [torch.empty((c[1].shape[0], c[0].N), dtype=torch.float32, device="cuda") for c in cases]
    first = []
    for (tw, x8, s_x, y64, ws), out in zip(cases, outs):
        binding.linear_tiled(x8, s_x, tw, out=out, out_dtype=binding.OUT_FP32, workspace=ws)
        torch.cuda.synchronize()
        worst, _ = fp32_gate(out.cpu().numpy(), y64, rel=2e-3)
        assert worst <= 2e-3, worst
        first.append(out.clone())
    # eager: 150 launches (more than two rounds of the 64 slots), alternating the two shapes
    for i in range(150):
        tw, x8, s_x, _, ws = cases[i & 1]
        outs[i & 1].fill_(float("nan"))
        binding.linear_tiled(x8, s_x, tw, out=outs[i & 1], out_dtype=binding.OUT_FP32, workspace=ws)
        if i % 37 == 0 or i >= 148:
            assert torch.equal(outs[i & 1], first[i & 1]), i
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    # one graph with 70 launches (slots repeat inside the graph), replayed several times
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(70):
                tw, x8, s_x, _, ws = cases[i & 1]
                binding.linear_tiled(x8, s_x, tw, out=outs[i & 1], out_dtype=binding.OUT_FP32, workspace=ws)
    torch.cuda.current_stream().wait_stream(side)
    for rep in range(5):
        for o in outs:
            o.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        for o, f in zip(outs, first):
            assert torch.equal(o, f), rep
    assert binding.query_device_status() == 0


def test_two_streams_issue_decode_launches_concurrently():
    # launches of two streams overlap on the device and share the placement table (different slots)
    a = _case(8, 14336, 4096, 11)
    b = _case(16, 18960, 2048, 13)
    outs = [torch.empty((c[1].shape[0], c[0].N), dtype=torch.float32, device="cuda") for c in (a, b)]
    first = []
    for (tw, x8, s_x, y64, ws), out in zip((a, b), outs):
        binding.linear_tiled(x8, s_x, tw, out=out, out_dtype=binding.OUT_FP32, workspace=ws)
        torch.cuda.synchronize()
        worst, _ = fp32_gate(out.cpu().numpy(), y64, rel=2e-3)
        assert worst <= 2e-3, worst
        first.append(out.clone())
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for s in streams:
        s.wait_stream(torch.cuda.current_stream())
    for rep in range(40):
        for i, (case, s) in enumerate(zip((a, b), streams)):
            tw, x8, s_x, _, ws = case
            with torch.cuda.stream(s):
                binding.linear_tiled(x8, s_x, tw, out=outs[i], out_dtype=binding.OUT_FP32, workspace=ws)
    for s in streams:
        torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    for o, f in zip(outs, first):
        assert torch.equal(o, f)
    assert binding.query_device_status() == 0


@pytest.mark.parametrize("shared_workspace", [False, True])
def test_chain_of_two_kernel_variants_never_waits_out_a_placement_hold(shared_workspace):
    # A chain that alternates a launch without a K cut (many output channels) and one with K cut
    # into chunks (few output channels) runs two instantiations of the decode kernel back to back,
    # each launch overlapping the next one's start.  Their placement slots must differ: when both
    # drew the same slot, candidates of one launch counted into the other's table and now and then
    # sat out the full hold limit (200 us), and worker indices could go missing.
    H, F, M = 4096, 14336, 1
    mk = lambda N, K, seed: binding.prepack_weight(
        *binding.quantize_weight_rtn(torch.from_numpy(inputs.make_weight(N, K, 0.02, seed)).cuda(), symmetric=True))
    wide, narrow = mk(2 * F, H, 71), mk(H, F, 72)
    x8a, sa = binding.quantize_act(bf16_dev(inputs.make_activation(M, H, 73)))
    x8b, sb = binding.quantize_act(bf16_dev(inputs.make_activation(M, F, 74)))
    ya = torch.empty((M, 2 * F), dtype=torch.bfloat16, device="cuda")
    yb = torch.empty((M, H), dtype=torch.bfloat16, device="cuda")
    wsa, wsb = binding.new_workspace(M, 2 * F, H, wide.fmt, "cuda"), binding.new_workspace(M, H, F, narrow.fmt, "cuda")
    if shared_workspace:    # allowed for calls issued one after the other on one stream
        wsb = wsa

    def chain():
        binding.linear_tiled(x8a, sa, wide, out=ya, workspace=wsa)
        binding.linear_tiled(x8b, sb, narrow, out=yb, workspace=wsb)

    chain()
    torch.cuda.synchronize()
    first = (ya.clone(), yb.clone())
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(6):
                chain()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for _ in range(60):
        g.replay()
    torch.cuda.synchronize()
    # what must hold whatever the placement did: no bounded wait ran out, every row range of every
    # launch was computed exactly once (a lost worker index leaves stale rows behind)
    assert binding.query_device_status() == 0
    ya2, yb2 = ya.clone(), yb.clone()
    ya.fill_(7.0)
    yb.fill_(7.0)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(ya, first[0]) and torch.equal(yb, first[1])
    assert torch.equal(ya2, first[0]) and torch.equal(yb2, first[1])


def test_launches_without_a_workspace_use_the_library_table_and_agree():
    # No (or too small a) workspace: the placement state is an entry of the library's own table and K
    # is never cut.  Results: equal bit for bit to the workspace path where that does not cut K
    # either (many output channels), within the output gate where it does (few output channels).
    tiny = torch.zeros((16,), dtype=torch.uint8, device="cuda")
    for M, N, K, cuts_k in ((4, 14336, 4096, False), (2, 4096, 14336, True)):
        tw, x8, s_x, y64, ws = _case(M, N, K, 31 + M)
        with_ws = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32, workspace=ws)
        outs = [binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32, workspace=tiny) for _ in range(70)]
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0
        worst, _ = fp32_gate(outs[0].cpu().numpy(), y64, rel=2e-3)
        assert worst <= 2e-3, worst
        assert all(torch.equal(o, outs[0]) for o in outs[1:])
        if not cuts_k:
            assert torch.equal(outs[0], with_ws)
        else:
            worst, _ = fp32_gate(with_ws.cpu().numpy(), y64, rel=2e-3)
            assert worst <= 2e-3, worst
