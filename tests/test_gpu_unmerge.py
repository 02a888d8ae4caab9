"""gsd_unmerge_tree on the GPU against the CPU oracle (bit-exact), and the unmerged tree run
through the verification kernels."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, attn_tensors, i32_tensor, out_to_f64
from helpers import verification_parents

pytestmark = pytest.mark.gpu


def run_gpu(tokens, ptr, idx, Ucap, max_depth, status=None):
    import paper_2407_16207_b200 as gsd
    out = gsd.gsd_unmerge_tree(i32_tensor(tokens, "cuda"), i32_tensor(ptr, "cuda"), i32_tensor(idx, "cuda"),
                               Ucap=Ucap, max_depth=max_depth, status=status)
    torch.cuda.synchronize()
    return [x.cpu().numpy() for x in out]


def check(tokens, ptr, idx, Ucap, max_depth, expect_full=None):
    want = oracle.unmerge_tree(tokens, ptr, idx, Ucap, max_depth)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = run_gpu(tokens, ptr, idx, Ucap, max_depth, status=status)
    for g, w in zip(got, want[:4]):
        assert np.array_equal(g, w)
    assert bool(int(status.item()) & 0x200) == want[4]
    assert int(status.item()) & ~0x200 == 0
    if expect_full is not None:
        assert want[4] == expect_full
    return want


@pytest.mark.parametrize("name,Ucap,max_depth,full", [
    ("tiny", 64, 99, None), ("tiny", 20, 99, True), ("llama7b", 4096, 99, None), ("llama7b", 512, 4, None),
    ("llama13b", 2048, 6, None), ("llama13b", 512, 99, True), ("llama70b", 512, 5, None),
    ("llama70b", 8192, 9, None)])
def test_generated_graphs_bit_exact(name, Ucap, max_depth, full):
    cfg = gi.CONFIGS[name]
    for trial in range(2):
        inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False, accept=False)
        check(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Ucap, max_depth, expect_full=full)


def grown_graph(seed, B=4, V=12, steps=6, k=3, tau=2, Ncap=256):
    """A token graph grown by the oracle's draft step from seeded draft logits over a small
    vocabulary (so that tau-grams really repeat), as parent lists of the verification DAG."""
    rng = np.random.default_rng(seed)
    tokens = np.full((B, Ncap), -1, np.int32); tokens[:, 0] = rng.integers(0, V, size=B)
    parent = np.full((B, Ncap), -1, np.int32); merge = np.full((B, Ncap), -1, np.int32)
    leaf = np.zeros((B, Ncap), np.uint8); prob = np.zeros((B, Ncap), np.float32); n = np.ones((B,), np.int32)
    F = 1
    fr = np.zeros((B, 1), np.int32); fl = np.ones((B,), np.int32)
    for _ in range(steps):
        lg = rng.standard_normal((B, F, V)).astype(np.float32) * 2
        tokens, parent, merge, leaf, prob, n, nf, nfl, _ = oracle.draft_expand(
            lg, fr, fl, tokens, parent, merge, leaf, prob, n, k=k, tau=tau, theta_prob=0.0, theta_sib=0.0)
        F = max(1, int(nfl.max()))
        fr = np.ascontiguousarray(nf[:, :F]); fl = nfl
        fr[fr < 0] = 0
    N = int(n.max())
    parents = []
    for b in range(B):
        ps = verification_parents(parent[b], merge[b], int(n[b]))
        parents.append(ps + [[] for _ in range(N - int(n[b]))])     # padding nodes: no parents, never reached
    ptr, idx = gi.parents_to_csr(parents)
    tok = np.where(tokens[:, :N] >= 0, tokens[:, :N], 0).astype(np.int32)
    return tok, ptr, idx, merge[:, :N], n


def test_graphs_grown_by_the_draft_step():
    merged = 0
    for seed in range(3):
        tok, ptr, idx, merge, n = grown_graph(seed)
        want = check(tok, ptr, idx, 2048, 12)
        merged += int((merge >= 0).sum())
        assert (want[3] >= n).all()                 # a tree node for every graph node that is reachable, and copies
    assert merged > 0                               # the graphs do contain merge edges


def test_duplicate_and_bad_parents():
    # node 2 lists parent 0 twice (one child copy), node 3 lists itself (ignored and flagged)
    ptr = np.array([[0, 0, 1, 3, 5]], np.int32)
    idx = np.array([[0, 0, 0, 3, 1]], np.int32)
    tok = np.array([[9, 8, 7, 6]], np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = run_gpu(tok, ptr, idx, 16, 9, status=status)
    assert int(status.item()) == 0x1
    cptr, cidx = gi.parents_to_csr([[[], [0], [0], [1]]], 5)
    want = oracle.unmerge_tree(tok, cptr, cidx, 16, 9)
    for g, w in zip(got, want[:4]):
        assert np.array_equal(g, w)


def test_unmerged_tree_through_the_verification_kernels():
    # the tree built on the device goes on to gsd_build_mask, gsd_verify_attn and gsd_accept (rows
    # gathered by tree_source); attention must match the oracle on the same tree, and acceptance
    # must pick the same tokens as on the graph itself
    import paper_2407_16207_b200 as gsd
    cfg = gi.VerifyConfig("t", 7, 2, 8, 2, 128, (40, 300), 48, 8, 3, 2, 500, 500, 0.8)
    inp = gi.make_inputs(cfg, 12)
    Ucap = 512
    t = {**attn_tensors(inp), **accept_tensors(inp)}
    tt, tp, ts, cnt = gsd.gsd_unmerge_tree(t["draft_tokens"], t["parent_ptr"], t["parent_idx"], Ucap=Ucap, max_depth=99)
    want = oracle.unmerge_tree(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Ucap, 99)
    assert not want[4] and np.array_equal(cnt.cpu().numpy(), want[3]) and (want[3] > cfg.N).all()
    # single-parent CSR of the tree, padded to Ucap nodes (padding nodes have no parent)
    n_tree = cnt.cpu().numpy()
    ptr = np.zeros((cfg.B, Ucap + 1), np.int32); idx = np.zeros((cfg.B, Ucap), np.int32)
    tp_h = tp.cpu().numpy()
    for b in range(cfg.B):
        e = 0
        for u in range(Ucap):
            ptr[b, u] = e
            if 0 < u < n_tree[b]:
                idx[b, e] = tp_h[b, u]; e += 1
        ptr[b, Ucap] = e
    d_ptr, d_idx = i32_tensor(ptr, "cuda"), i32_tensor(idx, "cuda")
    mask = gsd.gsd_build_mask(d_ptr, d_idx)
    src = ts.clamp(min=0).long()
    gather = lambda x: torch.gather(x, 1, src.view(cfg.B, Ucap, *([1] * (x.dim() - 2))).expand(-1, -1, *x.shape[2:])).contiguous()
    q, dk, dv, lg = gather(t["q"]), gather(t["draft_k"]), gather(t["draft_v"]), gather(t["logits"])
    out = gsd.gsd_verify_attn(q, t["k_cache"], t["v_cache"], dk, dv, mask, t["seq_lens"])
    toks, lens, nodes = gsd.gsd_accept(lg, tt.clamp(min=0), d_ptr, d_idx)
    torch.cuda.synchronize()
    src_h = src.cpu().numpy()
    take = lambda a: np.stack([a[b, src_h[b]] for b in range(cfg.B)])
    ref = oracle.attn(take(inp["q"]), inp["k_cache"], inp["v_cache"], take(inp["draft_k"]), take(inp["draft_v"]),
                      oracle.build_mask(ptr, idx), inp["seq_lens"])
    got = out_to_f64(out)
    for b in range(cfg.B):
        err = np.abs(got[b, :n_tree[b]] - ref[b, :n_tree[b]])
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
    t0, l0, n0, _ = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    assert np.array_equal(lens.cpu().numpy(), l0)
    for b in range(cfg.B):
        assert list(toks[b, :l0[b]].cpu().numpy()) == list(t0[b, :l0[b]])
        assert [int(src_h[b, u]) for u in nodes[b, :l0[b]].cpu().numpy()] == list(n0[b, :l0[b]])
