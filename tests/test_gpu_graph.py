"""A whole verification step captured into a CUDA graph and replayed: the library launches only on the
caller's stream, keeps no per-call device state that a replay would find stale (the split-KV counters are
cleared by the piece that merges), and so every replay reproduces the eager step bit for bit."""
import numpy as np
import pytest
import torch

import paper_2603_08088_b200 as tv
from workloads import CONFIGS, make_case
from gpu_util import to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ci,over", [(4, dict(B=6, L=3, Hq=8, Hkv=2, S_lo=100, S_hi=1500, Scap=1600, V=4096)),
                                     (1, dict(Hq=8, Hkv=8, S_lo=2048, S_hi=2048, Scap=2304, V=2048, L=2))])
def test_step_replayed_from_a_cuda_graph_equals_the_eager_step(ci, over):
    cfg = CONFIGS[ci].scaled(**over)
    case = to_device(make_case(cfg, seed=99 + ci))
    P, Dp1 = case["retrieve"].shape[1], cfg.D + 1
    buf = tv.StepBuffers(cfg.L, cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.Scap, cfg.V, P, Dp1, device="cuda", want_lse=True)
    scale = cfg.d ** -0.5
    saved = {k: case[k].clone() for k in ("prefix_len", "k_cache", "v_cache")}

    def restore():
        for k, v in saved.items():
            case[k].copy_(v)

    def snapshot():
        torch.cuda.synchronize()
        return {"out": buf.out.clone(), "lse": buf.lse.clone(), "accept_len": buf.accept_len.clone(),
                "accepted_nodes": buf.accepted_nodes.clone(), "next_token": buf.next_token.clone(),
                "prefix_len": case["prefix_len"].clone(), "k_cache": case["k_cache"].clone(),
                "v_cache": case["v_cache"].clone(), "status": buf.status.clone()}

    tv.verify_step(case, buf, scale, retrieve=case["retrieve"])           # eager (also the warm-up the capture needs)
    want = snapshot()
    assert (want["status"] == 0).all()
    restore()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        tv.verify_step(case, buf, scale, retrieve=case["retrieve"])       # once more on the side stream before capturing
        torch.cuda.synchronize()
        restore()
        with torch.cuda.graph(graph, stream=stream):
            tv.verify_step(case, buf, scale, retrieve=case["retrieve"])
    torch.cuda.current_stream().wait_stream(stream)
    for replay in range(3):
        restore()
        buf.out.zero_()
        buf.accept_len.fill_(-1)
        graph.replay()
        got = snapshot()
        for k in want:
            a, b = got[k], want[k]
            if a.dtype == torch.bfloat16:
                a, b = a.view(torch.int16), b.view(torch.int16)
            assert torch.equal(a, b), f"replay {replay}: {k} differs from the eager step"
