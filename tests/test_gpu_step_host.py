"""The host-buffer step: same results as the device calls, through one C-ABI call."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, attn_tensors, out_to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "llama7b"])
def test_step_from_host_buffers(name):
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg)
    h = {**attn_tensors(inp, "cpu"), **accept_tensors(inp, "cpu")}
    h = {k: v.pin_memory() for k, v in h.items()}
    Ecap = h["parent_idx"].shape[1]
    nbytes = gsd.gsd_verify_step_host_arena_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D,
                                                  inp["Lmax"], cfg.V, Ecap, cfg.N)
    assert nbytes > 0
    arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        out, toks, lens, nodes, status = gsd.gsd_verify_step_host(
            h["q"], h["k_cache"], h["v_cache"], h["draft_k"], h["draft_v"], h["ancestor_mask"],
            h["seq_lens"], h["logits"], h["draft_tokens"], h["parent_ptr"], h["parent_idx"], arena)
        assert status == 0
        want = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                           inp["ancestor_mask"], inp["seq_lens"])
        err = np.abs(out_to_f64(out) - want)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
        wt, wl, wn, _ = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"],
                                      inp["parent_idx"])
        assert np.array_equal(toks.numpy(), wt) and np.array_equal(lens.numpy(), wl)
        assert np.array_equal(nodes.numpy(), wn)
    with pytest.raises(gsd.GsdError):
        gsd.gsd_verify_step_host(
            h["q"], h["k_cache"], h["v_cache"], h["draft_k"], h["draft_v"], h["ancestor_mask"],
            h["seq_lens"], h["logits"], h["draft_tokens"], h["parent_ptr"], h["parent_idx"],
            arena[:1024])


@pytest.mark.parametrize("num_splits", [-1, -2])
def test_step_from_host_buffers_with_plans_made_on_the_device(num_splits):
    # the planning kernel reads seq_lens from the arena, behind the copy of the same call
    import paper_2407_16207_b200 as gsd
    cfg = gi.VerifyConfig("h", 7, 3, 8, 2, 128, (10, 700), 70, 9, 3, 2, 500, 500, 0.6)
    inp = gi.make_inputs(cfg, 4)
    h = {**attn_tensors(inp, "cpu"), **accept_tensors(inp, "cpu")}
    h = {k: v.pin_memory() for k, v in h.items()}
    Ecap = h["parent_idx"].shape[1]
    nbytes = gsd.gsd_verify_step_host_arena_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, inp["Lmax"], cfg.V, Ecap, cfg.N,
                                                  num_splits=num_splits, kernel=2)
    arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        out, toks, lens, nodes, status = gsd.gsd_verify_step_host(
            h["q"], h["k_cache"], h["v_cache"], h["draft_k"], h["draft_v"], h["ancestor_mask"],
            h["seq_lens"], h["logits"], h["draft_tokens"], h["parent_ptr"], h["parent_idx"], arena,
            num_splits=num_splits, kernel=2)
        assert status == 0
        want = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                           inp["ancestor_mask"], inp["seq_lens"])
        err = np.abs(out_to_f64(out) - want)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
        wt, wl, wn, _ = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        assert np.array_equal(toks.numpy(), wt) and np.array_equal(lens.numpy(), wl) and np.array_equal(nodes.numpy(), wn)
