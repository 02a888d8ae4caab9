"""Out-of-bounds writes, looked for without a sanitizer: every output and every scratch buffer of
every call sits inside a larger allocation whose margins hold a sentinel; after the call the
margins must be untouched (and the results still match the oracle).  Shapes are chosen so that
the tiles of the kernels overhang the tensors: node counts that are no multiple of a row tile,
ragged prefixes, forced key-range splits."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, attn_tensors, i32_tensor, out_to_f64

pytestmark = pytest.mark.gpu

MARGIN = 4096        # bytes on each side


class Guarded:
    """A tensor of the given shape and dtype inside a byte buffer with sentinel margins."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.n = n
        self.buf = torch.full((n + 2 * MARGIN,), 0xA5, dtype=torch.uint8, device="cuda")
        self.t = self.buf[MARGIN:MARGIN + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.copy_(fill)

    def intact(self):
        return bool((self.buf[:MARGIN] == 0xA5).all()) and bool((self.buf[MARGIN + self.n:] == 0xA5).all())


def all_intact(*guards):
    torch.cuda.synchronize()
    return all(g.intact() for g in guards)


@pytest.mark.parametrize("kernel,splits", [(2, 0), (2, 3), (2, -1), (2, -2), (1, 0), (1, 3)])
def test_attention_output_and_workspace(kernel, splits):
    import paper_2407_16207_b200 as gsd
    # R = N * G = 400 stacked rows: the last 128-row tile is partial, N is no multiple of 128 / G
    cfg = gi.VerifyConfig("c", 8, 2, 16, 2, 128, (70, 333), 50, 8, 3, 2, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 21, accept=False, pad_fill="nan")
    t = attn_tensors(inp)
    out = Guarded(t["q"].shape, torch.bfloat16)
    need = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, inp["Lmax"], splits, kernel)
    ws = Guarded((max(need, 256),), torch.uint8)
    gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], t["ancestor_mask"],
                        t["seq_lens"], out=out.t, kernel=kernel, num_splits=splits, workspace=ws.t)
    assert all_intact(out, ws)
    want = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                       inp["ancestor_mask"], inp["seq_lens"])
    err = np.abs(out_to_f64(out.t) - want)
    assert err.max() <= 1e-2 and err.mean() <= 1e-3


def test_attention_llama7b_tcgen05_tma_stores():
    # the configuration the automatic choice sends to the tcgen05 kernel with forced splits: TMA
    # tile stores of the epilogue and the fp32 partial results of the split pass
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, accept=False)
    t = attn_tensors(inp)
    out = Guarded(t["q"].shape, torch.bfloat16)
    need = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, inp["Lmax"])
    ws = Guarded((max(need, 256),), torch.uint8)
    gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], t["ancestor_mask"],
                        t["seq_lens"], out=out.t, workspace=ws.t)
    assert all_intact(out, ws)


def test_accept_and_accept_sampled():
    import paper_2407_16207_b200 as gsd
    cfg = gi.VerifyConfig("c", 8, 3, 1, 1, 64, 8, 37, 7, 3, 2, 1003, 1003, 0.7)
    inp = gi.make_inputs(cfg, 5, attn=False)
    t = accept_tensors(inp)
    B, N, Tcap = cfg.B, cfg.N, 9
    toks, lens, nodes = Guarded((B, Tcap), torch.int32), Guarded((B,), torch.int32), Guarded((B, Tcap), torch.int32)
    ws = Guarded((gsd.gsd_accept_workspace_bytes(B, N),), torch.uint8)
    gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"], Tcap=Tcap,
                   workspace=ws.t, out=(toks.t, lens.t, nodes.t))
    assert all_intact(toks, lens, nodes, ws)
    want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Tcap=Tcap)
    assert np.array_equal(toks.t.cpu().numpy(), want[0]) and np.array_equal(lens.t.cpu().numpy(), want[1])

    rng = np.random.default_rng(1)
    q = torch.from_numpy(rng.uniform(0.05, 1, size=(B, N)).astype(np.float32)).cuda()
    u = torch.from_numpy(rng.uniform(0, 1, size=(B, N)).astype(np.float32)).cuda()
    us = torch.from_numpy(rng.uniform(0, 1, size=(B,)).astype(np.float32)).cuda()
    dl = torch.from_numpy(rng.standard_normal(inp["logits"].shape).astype(np.float32)).cuda()
    toks2, lens2, nodes2 = Guarded((B, Tcap), torch.int32), Guarded((B,), torch.int32), Guarded((B, Tcap), torch.int32)
    ws2 = Guarded((gsd.gsd_accept_sampled_workspace_bytes(B, N),), torch.uint8)
    gsd.gsd_accept_sampled(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"], q, u, us,
                           draft_logits=dl, Tcap=Tcap, workspace=ws2.t, out=(toks2.t, lens2.t, nodes2.t))
    assert all_intact(toks2, lens2, nodes2, ws2)


def test_commit_kv_build_mask_and_unmerge():
    import paper_2407_16207_b200 as gsd
    cfg = gi.VerifyConfig("c", 8, 2, 4, 2, 64, (20, 60), 21, 5, 3, 2, 50, 50, 0.8)
    inp = gi.make_inputs(cfg, 9)
    t = {**attn_tensors(inp), **accept_tensors(inp)}
    B, N, Lmax = cfg.B, cfg.N, inp["Lmax"]
    # the cache is full for the longest sequence: rows past Lmax must be dropped, not written
    kc = Guarded(t["k_cache"].shape, torch.bfloat16, t["k_cache"])
    vc = Guarded(t["v_cache"].shape, torch.bfloat16, t["v_cache"])
    sl = Guarded((B,), torch.int32, t["seq_lens"])
    toks, lens, nodes = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gsd.gsd_commit_kv(kc.t, vc.t, t["draft_k"], t["draft_v"], nodes, lens, sl.t, status=status)
    assert all_intact(kc, vc, sl)
    assert int(status.item()) & 0x20                      # the full sequence overflowed and said so
    assert int(sl.t.max().item()) <= Lmax

    mask = Guarded((B, N, (N + 31) // 32), torch.int32)
    gsd.gsd_build_mask(t["parent_ptr"], t["parent_idx"], out=mask.t)
    assert all_intact(mask)
    assert np.array_equal(mask.t.cpu().numpy().view(np.uint32), inp["ancestor_mask"])

    Ucap = 77
    outs = [Guarded((B, Ucap), torch.int32) for _ in range(3)] + [Guarded((B,), torch.int32)]
    gsd.gsd_unmerge_tree(t["draft_tokens"], t["parent_ptr"], t["parent_idx"], Ucap=Ucap, max_depth=99,
                         out=tuple(g.t for g in outs))
    assert all_intact(*outs)
    want = oracle.unmerge_tree(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Ucap, 99)
    for g, w in zip(outs, want[:4]):
        assert np.array_equal(g.t.cpu().numpy(), w)


def test_draft_expand():
    import paper_2407_16207_b200 as gsd
    B, F, V, Ncap, k = 3, 5, 1003, 40, 4
    rng = np.random.default_rng(2)
    lg = torch.from_numpy(rng.standard_normal((B, F, V)).astype(np.float32)).cuda()
    n0 = 23                                                   # 23 + 5 * 4 = 43 > Ncap: the capacity cuts the last children
    tokens = Guarded((B, Ncap), torch.int32, torch.from_numpy(rng.integers(0, V, size=(B, Ncap)).astype(np.int32)))
    par_h = np.tile(np.arange(-1, Ncap - 1, dtype=np.int32), (B, 1))
    parent = Guarded((B, Ncap), torch.int32, torch.from_numpy(par_h))
    merge = Guarded((B, Ncap), torch.int32, torch.full((B, Ncap), -1, dtype=torch.int32))
    leaf = Guarded((B, Ncap), torch.uint8, torch.zeros((B, Ncap), dtype=torch.uint8))
    prob = Guarded((B, Ncap), torch.float32, torch.zeros((B, Ncap)))
    num = Guarded((B,), torch.int32, torch.full((B,), n0, dtype=torch.int32))
    fr = torch.from_numpy(np.tile(np.arange(F, dtype=np.int32) + 3, (B, 1))).cuda()
    fl = torch.full((B,), F, dtype=torch.int32, device="cuda")
    nf, nfl = Guarded((B, F * k), torch.int32), Guarded((B,), torch.int32)
    p = gsd.binding.DraftParams(B, F, V, Ncap, k, 2, 0.0, 0.0)
    import ctypes
    need = int(gsd.lib().gsd_draft_expand_workspace_bytes(ctypes.byref(p)))
    ws = Guarded((need,), torch.uint8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gsd.gsd_draft_expand(lg, fr, fl, tokens.t, parent.t, merge.t, leaf.t, prob.t, num.t, k=k, tau=2,
                         theta_prob=0.0, theta_sib=0.0, workspace=ws.t, status=status, out=(nf.t, nfl.t))
    assert all_intact(tokens, parent, merge, leaf, prob, num, nf, nfl, ws)
    assert int(status.item()) == 0x80 and int(num.t.max().item()) == Ncap
