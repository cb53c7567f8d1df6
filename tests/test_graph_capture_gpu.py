"""The forward-path calls allocate nothing and never synchronise, so a sequence of them can be recorded
into a CUDA graph and replayed: the replay must write the same bytes as the eager calls, also after
the input buffers' contents have changed."""
import pytest
import torch

from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


def test_permute_forward_unpermute_and_fused_replay_from_a_graph():
    H, W, tile, hs, nt, B, heads = 32, 32, 128, 4, 77, 1, 3
    S = nt + H * W
    g = torch.Generator().manual_seed(4242)
    q, k, v = (torch.randn((B, heads, S, 128), generator=g).bfloat16().cuda() for _ in range(3))
    plans = [hb.Plan(H, W, tile, o, hs, nt) for o in (0, 32, 64, 96)]
    try:
        for p in plans:
            p.bind_like(q)
        qp, kp, vp, a, b, out, fused = (torch.empty_like(q) for _ in range(7))

        def step(stream):
            # entry gathers, four layers with different offsets, exit gather; and the one-launch form
            plans[0].permute(q, qp, stream=stream)
            plans[0].permute(k, kp, stream=stream)
            plans[0].permute(v, vp, stream=stream)
            plans[0].forward(qp, kp, vp, a, stream=stream)
            plans[1].forward(a, kp, vp, b, stream=stream)
            plans[2].forward(b, kp, vp, a, stream=stream)
            plans[3].forward(a, kp, vp, b, stream=stream)
            plans[3].unpermute(b, out, stream=stream)
            plans[1].forward_fused(q, k, v, fused, in_original=True, out_original=True, stream=stream)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step(side)                      # warm-up outside the capture
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step(side)
        for trial in range(3):
            # new contents in the same buffers
            for t in (q, k, v):
                t.copy_(torch.randn(t.shape, generator=g).bfloat16())
            step(torch.cuda.current_stream())
            torch.cuda.synchronize()
            ref_out, ref_fused = out.clone(), fused.clone()
            out.fill_(float("nan"))
            fused.fill_(float("nan"))
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16)), trial
            assert torch.equal(fused.view(torch.int16), ref_fused.view(torch.int16)), trial
        for p in plans:
            assert p.status() == 0
    finally:
        for p in plans:
            p.destroy()
