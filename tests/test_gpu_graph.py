"""The device-pointer calls only enqueue work on the caller's stream, so a whole verification
step can be captured in a CUDA graph and replayed; the replay must reproduce the eager results."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
from gpu_util import accept_tensors, attn_tensors

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,num_splits", [("llama7b", 0), ("llama13b", 0), ("llama13b", -1), ("llama13b", -2)])
def test_step_replays_from_a_cuda_graph(name, num_splits):
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg)
    t = {**attn_tensors(inp), **accept_tensors(inp)}
    B, N = cfg.B, cfg.N
    out = torch.empty_like(t["q"])
    ws = torch.empty(max(256, gsd.gsd_verify_attn_workspace_bytes(B, N, cfg.Hq, cfg.Hkv, cfg.D, inp["Lmax"], num_splits)),
                     dtype=torch.uint8, device="cuda")
    ws_acc = torch.empty(gsd.gsd_accept_workspace_bytes(B, N), dtype=torch.uint8, device="cuda")
    acc = (torch.empty((B, N), dtype=torch.int32, device="cuda"), torch.empty((B,), dtype=torch.int32, device="cuda"),
           torch.empty((B, N), dtype=torch.int32, device="cuda"))
    mask_out = torch.empty_like(t["ancestor_mask"])

    def step():
        gsd.gsd_build_mask(t["parent_ptr"], t["parent_idx"], out=mask_out)
        gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], mask_out,
                            t["seq_lens"], out=out, workspace=ws, num_splits=num_splits)
        gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"], workspace=ws_acc, out=acc)

    step()                                   # eager (also the first-call set-up of the library)
    torch.cuda.synchronize()
    want_out = out.clone()
    want_acc = [x.clone() for x in acc]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    out.zero_()
    for x in acc:
        x.fill_(-7)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want_out)
    for x, y in zip(acc, want_acc):
        assert torch.equal(x, y)
    assert torch.equal(mask_out, t["ancestor_mask"])
