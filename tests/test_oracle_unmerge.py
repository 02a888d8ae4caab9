"""Pins of the oracle's unmerging of the token graph into a tree (Sec. 5.4, Fig. 4: the
successors of a redundant node are replicated from the node it was merged into, then the tree
is verified as in tree-structured decoding)."""
import numpy as np
import torch
import torch.nn.functional as F

import gsd_inputs as gi
import oracle
from helpers import root_paths, verification_parents
from test_oracle_draft import forcing_logits, fresh, grow


def unmerge(parents, tokens, Ucap, max_depth):
    ptr, idx = gi.parents_to_csr([parents])
    tt, tp, ts, cnt, full = oracle.unmerge_tree(np.array([tokens], np.int32), ptr, idx, Ucap, max_depth)
    n = int(cnt[0])
    assert (tt[0, n:] == -1).all() and (tp[0, n:] == -1).all() and (ts[0, n:] == -1).all()
    return list(tt[0, :n]), list(tp[0, :n]), list(ts[0, :n]), full


def test_worked_example_from_a_grown_graph():
    # the graph of the redundancy example with tau = 2: root 5 -> 1, 2; node 1 -> 3, 4;
    # node 2 -> 3, 7; node 3 -> 8, 9; node 5 (token 3) -> 8, 6, where node 9 = (3, 8) under node 5
    # repeats (3, 8) of node 7 and is merged into it.  Node 7 gets children 11, 12 in one more step.
    V = 12
    st = fresh(1, 32)
    st, _, _, _ = grow(st, forcing_logits([[1, 2]], V), [[0]], 2, 2)
    st, _, _, _ = grow(st, forcing_logits([[3, 4], [3, 7]], V), [[1, 2]], 2, 2)
    st, nf, nfl, _ = grow(st, forcing_logits([[8, 9], [8, 6]], V), [[3, 5]], 2, 2)
    assert int(st[2][0, 9]) == 7 and list(nf[0, :nfl[0]]) == [7, 8, 10]
    st, _, _, _ = grow(st, forcing_logits([[10, 11], [0, 1], [0, 2]], V), [[7, 8, 10]], 2, 2)
    tok, par, mrg, leaf, prob, n = st
    n = int(n[0])
    assert n == 17 and list(par[0, 11:13]) == [7, 7]
    parents = verification_parents(par[0], mrg[0], n)
    assert parents[11] == [7, 9] and parents[12] == [7, 9]       # the merged node re-uses node 7's successors
    tt, tp, ts, full = unmerge(parents, list(tok[0, :n]), 64, 10)
    # the tree: the 17 nodes plus one copy each of nodes 11 and 12 under node 9
    assert not full and len(tt) == 19
    assert ts[:11] == list(range(11))                          # levels 0-3 are already a tree in level order
    # level 4 in the order of the parents 7, 8, 9 (the merged node: copies of 11, 12), 10
    assert ts[11:] == [11, 12, 13, 14, 11, 12, 15, 16]
    assert tp[11:] == [7, 7, 8, 8, 9, 9, 10, 10]
    assert tt[15] == tok[0, 11] and tt[16] == tok[0, 12]


def test_a_tree_in_level_order_is_left_as_it_is():
    cfg = gi.VerifyConfig("t", 7, 1, 1, 1, 64, 4, 40, 6, 3, 1, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 3, attn=False, accept=False)
    parents = inp["parents"][0]
    tt, tp, ts, full = unmerge(parents, list(inp["draft_tokens"][0]), 64, 99)
    # level order, children grouped by parent: the generator's numbering may differ inside a level,
    # but the map is a bijection that keeps tokens, parents and levels
    assert sorted(ts) == list(range(cfg.N)) and not full
    for u in range(1, cfg.N):
        assert parents[ts[u]] == [ts[tp[u]]] and tp[u] < u
        assert tt[u] == inp["draft_tokens"][0, ts[u]]
    lv = [inp["levels"][0][s] for s in ts]
    assert lv == sorted(lv)


def test_every_root_path_appears_exactly_once():
    for seed, depth_cap in ((1, 99), (2, 99), (3, 4)):
        cfg = gi.VerifyConfig("t", 7, 1, 1, 1, 64, 4, 24, 6, 3, 2, 8, 8, 0.5)
        inp = gi.make_inputs(cfg, seed, attn=False, accept=False)
        parents = inp["parents"][0]
        want = root_paths(parents, depth_cap)
        tt, tp, ts, full = unmerge(parents, list(inp["draft_tokens"][0]), 4096, depth_cap)
        assert not full
        got = []
        for u in range(len(tt)):
            path, x = [], u
            while x >= 0:
                path.append(ts[x]); x = tp[x]
            got.append(tuple(reversed(path)))
        assert len(got) == len(want) and sorted(got) == sorted(want)
        assert len(set(got)) == len(got)
        # numbering: level by level, inside a level by (parent's tree index, copied node id)
        key = [(len(p), tp[u], ts[u]) for u, p in enumerate(got)]
        assert key == sorted(key)


def test_node_count_of_a_chain_of_diamonds():
    # k diamonds in a row (a -> {b, c} -> d): 2^i paths reach the i-th joint, so the tree has
    # 1 + sum_i (2^i + 2^i) + ... nodes: joints 2^i copies each, the two middle nodes 2^(i-1) each
    k = 5
    parents = [[]]
    for i in range(k):
        j = 3 * i                      # joint node of diamond i
        parents += [[j], [j], [j + 1, j + 2]]
    tt, tp, ts, full = unmerge(parents, list(range(len(parents))), 4096, 99)
    want = 1 + sum(2 * 2 ** i + 2 ** (i + 1) for i in range(k))
    assert len(tt) == want and not full
    assert ts.count(3 * k) == 2 ** k


def test_depth_limit_and_capacity():
    tt, tp, ts, full = unmerge([[], [0]], [4, 4], 16, 0)
    assert tt == [4] and tp == [-1]                      # max_depth 0: the root alone
    cfg = gi.VerifyConfig("t", 7, 1, 1, 1, 64, 4, 30, 8, 3, 3, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 5, attn=False, accept=False)
    parents = inp["parents"][0]
    all_paths = root_paths(parents, 99)
    for d in (1, 3, 5):
        tt, tp, ts, full = unmerge(parents, list(inp["draft_tokens"][0]), 1 << 16, d)
        assert len(tt) == len([p for p in all_paths if len(p) - 1 <= d])
    cap = 50
    assert len(all_paths) > cap
    tt, tp, ts, full = unmerge(parents, list(inp["draft_tokens"][0]), cap, 99)
    big = unmerge(parents, list(inp["draft_tokens"][0]), 1 << 16, 99)
    assert full and len(tt) == cap
    assert (tt, tp, ts) == (big[0][:cap], big[1][:cap], big[2][:cap])     # a prefix of the level order


def test_acceptance_on_the_tree_equals_acceptance_on_the_graph():
    # a tree copy carries its source node's logits row: every accepted path of the graph is an
    # accepted path of the tree and vice versa, so length and tokens agree (Sec. 5.4: "the same
    # verification procedure as used in TSD")
    cfg = gi.VerifyConfig("t", 7, 3, 1, 1, 64, 4, 28, 7, 3, 2, 50, 50, 0.8)
    for seed in range(4):
        inp = gi.make_inputs(cfg, 20 + seed, attn=False)
        t0, l0, n0, _ = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        Ucap = 2048
        tt, tp, ts, cnt, full = oracle.unmerge_tree(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Ucap, 99)
        assert not full
        for b in range(cfg.B):
            n = int(cnt[b])
            parents = [[] if u == 0 else [int(tp[b, u])] for u in range(n)]
            ptr, idx = gi.parents_to_csr([parents])
            t1, l1, n1, _ = oracle.accept(inp["logits"][b, ts[b, :n]][None], tt[b, :n][None], ptr, idx, visit_cap=10 ** 6)
            assert l1[0] == l0[b]
            assert list(t1[0, :l1[0]]) == list(t0[b, :l0[b]])
            assert [int(ts[b, u]) for u in n1[0, :l1[0]]] == list(n0[b, :l0[b]])


def test_attention_on_the_unmerged_tree_is_per_path_sequential_decoding():
    # each tree node sees the prefix and its own root path only (tree attention, Sec. 4.1)
    cfg = gi.VerifyConfig("t", 7, 1, 4, 2, 64, 9, 14, 4, 3, 2, 8, 8, 0.5)
    inp = gi.make_inputs(cfg, 4, accept=False)
    tt, tp, ts, cnt, full = oracle.unmerge_tree(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], 256, 99)
    n = int(cnt[0])
    assert n > cfg.N and not full
    parents = [[] if u == 0 else [int(tp[0, u])] for u in range(n)]
    mask = gi.closure_mask(parents)[None]
    src = ts[0, :n]
    q, dk, dv = inp["q"][:, src], inp["draft_k"][:, src], inp["draft_v"][:, src]
    out = oracle.attn(q, inp["k_cache"], inp["v_cache"], dk, dv, mask, inp["seq_lens"])
    f64 = lambda a: torch.from_numpy(gi.bf16_bits_to_f32(a).astype(np.float64))
    L = cfg.L
    for u in range(n):
        path, x = [], u
        while x >= 0:
            path.append(x); x = int(tp[0, x])
        path = path[::-1]
        ii = torch.tensor(path)
        k = torch.cat([f64(inp["k_cache"][0, :L]), f64(dk[0])[ii]]).repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        v = torch.cat([f64(inp["v_cache"][0, :L]), f64(dv[0])[ii]]).repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        qfull = torch.zeros(cfg.Hq, L + len(path), cfg.D, dtype=torch.float64)
        qfull[:, L:] = f64(q[0])[ii].permute(1, 0, 2)
        ref = F.scaled_dot_product_attention(qfull[None], k[None], v[None], is_causal=True)[0, :, -1].numpy()
        assert np.allclose(out[0, u], ref, rtol=0, atol=1e-12)
