"""The index-checking build of the library (libgsd_check.so, compiled with -DGSD_BOUNDS_CHECK)
run over every call: its kernels check the indices they form into global memory (key and node
positions, plan slots, graph capacities, output capacities) and would OR GSD_DEV_BOUNDS into the
status word instead of touching memory outside a tensor.  On well-formed inputs the bit must
stay clear and the results must be the ordinary ones.  This stands in for a memory sanitizer."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, attn_tensors, out_to_f64

pytestmark = pytest.mark.gpu

GSD_DEV_BOUNDS = 0x400


@pytest.fixture()
def checked_lib():
    """Points the binding at the checking build for one test, then back."""
    from paper_2407_16207_b200 import binding, build
    path = build.build(checked=True)
    saved = (binding._lib, binding._LIB_PATH)
    binding._lib, binding._LIB_PATH = None, path
    try:
        import paper_2407_16207_b200 as gsd
        assert gsd.lib()._name == path
        yield gsd
    finally:
        binding._lib, binding._LIB_PATH = saved


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b"])
def test_every_call_keeps_its_indices_inside(checked_lib, name):
    gsd = checked_lib
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg)
    t = {**attn_tensors(inp), **accept_tensors(inp)}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want_attn = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                            inp["ancestor_mask"], inp["seq_lens"])
    for kernel, splits in ((0, 0), (1, 0), (1, 3), (2, 0), (2, 3), (2, -1), (2, -2)):
        if kernel == 2 and cfg.D != 128:
            continue
        out = gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], t["ancestor_mask"],
                                  t["seq_lens"], kernel=kernel, num_splits=splits, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (kernel, splits)
        err = np.abs(out_to_f64(out) - want_attn)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
    toks, lens, nodes = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"], status=status)
    want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    assert np.array_equal(toks.cpu().numpy(), want[0]) and np.array_equal(nodes.cpu().numpy(), want[2])
    rng = np.random.default_rng(3)
    B, N = cfg.B, cfg.N
    q = torch.from_numpy(rng.uniform(0.05, 1, size=(B, N)).astype(np.float32)).cuda()
    u = torch.from_numpy(rng.uniform(0, 1, size=(B, N)).astype(np.float32)).cuda()
    us = torch.from_numpy(rng.uniform(0.1, 0.9, size=(B,)).astype(np.float32)).cuda()
    dl = torch.from_numpy((inp["logits"] + rng.standard_normal(inp["logits"].shape).astype(np.float32)).astype(np.float32)).cuda()
    gsd.gsd_accept_sampled(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"], q, u, us,
                           draft_logits=dl, status=status)
    mask = gsd.gsd_build_mask(t["parent_ptr"], t["parent_idx"], status=status)
    assert np.array_equal(mask.cpu().numpy().view(np.uint32), inp["ancestor_mask"])
    grow = cfg.depth + 1
    pad = torch.zeros((B, grow, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device="cuda")
    kc = torch.cat([t["k_cache"], pad], dim=1).contiguous()
    vc = torch.cat([t["v_cache"], pad], dim=1).contiguous()
    sl = t["seq_lens"].clone()
    gsd.gsd_commit_kv(kc, vc, t["draft_k"], t["draft_v"], nodes, lens, sl, status=status)
    tt, tp, ts, cnt = gsd.gsd_unmerge_tree(t["draft_tokens"], t["parent_ptr"], t["parent_idx"], Ucap=300, max_depth=5,
                                           status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & ~0x200 == 0           # (the tree capacity may be reached: that is not an index error)
    status.zero_()
    # one growth step of a draft graph over the same vocabulary
    V, F, Ncap, k = cfg.V, 6, 64, 4
    lg = torch.from_numpy(rng.standard_normal((B, F, V)).astype(np.float32)).cuda()
    tokens = torch.zeros((B, Ncap), dtype=torch.int32, device="cuda")
    parent = torch.arange(-1, Ncap - 1, dtype=torch.int32, device="cuda").repeat(B, 1).contiguous()
    merge = torch.full((B, Ncap), -1, dtype=torch.int32, device="cuda")
    leaf = torch.zeros((B, Ncap), dtype=torch.uint8, device="cuda")
    prob = torch.zeros((B, Ncap), dtype=torch.float32, device="cuda")
    num = torch.full((B,), 30, dtype=torch.int32, device="cuda")
    fr = torch.arange(F, dtype=torch.int32, device="cuda").repeat(B, 1).contiguous()
    fl = torch.full((B,), F, dtype=torch.int32, device="cuda")
    gsd.gsd_draft_expand(lg, fr, fl, tokens, parent, merge, leaf, prob, num, k=k, tau=2, theta_prob=0.0,
                         theta_sib=0.0, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & GSD_DEV_BOUNDS == 0
    assert int(num.max().item()) == 30 + F * k
