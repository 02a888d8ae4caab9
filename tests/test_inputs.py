"""The synthetic input generator: structure of the draft DAGs and of the tensors."""
import numpy as np
import pytest

import gsd_inputs as gi


def test_full_kary_tree_level_sizes_match_closed_form():
    # a full tree of depth gamma and out-degree k holds (k^(gamma+1)-1)/(k-1) nodes (Sec. 4)
    for k, gamma in [(2, 4), (3, 3), (4, 3)]:
        n = (k ** (gamma + 1) - 1) // (k - 1)
        assert gi.level_sizes(n, gamma, k) == [k ** l for l in range(gamma + 1)]
        with pytest.raises(ValueError):
            gi.level_sizes(n + 1, gamma, k)


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
def test_dag_structure(name):
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg, attn=False, accept=False)
    assert inp["draft_tokens"].shape == (cfg.B, cfg.N)
    for b in range(cfg.B):
        parents, level = inp["parents"][b], inp["levels"][b]
        assert parents[0] == [] and max(level) == cfg.depth
        children = gi.children_of(parents)
        assert max(len(c) for c in children) <= cfg.kmax
        for v in range(1, cfg.N):
            assert 1 <= len(parents[v]) <= cfg.pmax
            assert len(set(parents[v])) == len(parents[v])
            assert all(p < v and level[p] == level[v] - 1 for p in parents[v])
        ptr, idx = inp["parent_ptr"][b], inp["parent_idx"][b]
        for v in range(cfg.N):
            assert list(idx[ptr[v]:ptr[v + 1]]) == parents[v]


def test_mask_is_reflexive_transitive_closure():
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, attn=False, accept=False)
    parents = inp["parents"][0]
    # reachability by explicit upward search, node by node
    for v in range(cfg.N):
        seen, todo = {v}, [v]
        while todo:
            for p in parents[todo.pop()]:
                if p not in seen:
                    seen.add(p)
                    todo.append(p)
        row = inp["ancestor_mask"][0, v]
        got = {j for j in range(cfg.W * 32) if (int(row[j // 32]) >> (j % 32)) & 1}
        assert got == seen


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 1.00390625, 1.01171875, 3.0e37], dtype=np.float32)
    bits = gi.f32_to_bf16_bits(x)
    back = gi.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: round to even mantissa (1.0)
    assert back[0] == 1.0 and back[1] == -2.5 and back[2] == 1.0
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 (odd) and 1 + 2^-6 (even): goes up
    assert back[3] == np.float32(1.015625)
    assert np.isfinite(back[4])


def test_seeded_and_distinct():
    cfg = gi.CONFIGS["tiny"]
    a, b, c = gi.make_inputs(cfg, 7), gi.make_inputs(cfg, 7), gi.make_inputs(cfg, 8)
    for key in ("q", "k_cache", "logits", "draft_tokens", "ancestor_mask"):
        assert np.array_equal(a[key], b[key])
    assert not np.array_equal(a["q"], c["q"])


def test_ragged_prefix_padding_fill():
    cfg = gi.CONFIGS["llama13b"]
    cfg = gi.VerifyConfig(**{**cfg.__dict__, "L": (10, 40), "Hq": 2, "Hkv": 2, "N": 16,
                             "depth": 4, "V": 50, "vtok": 50})
    inp = gi.make_inputs(cfg, pad_fill="nan")
    L = inp["seq_lens"]
    assert inp["Lmax"] == L.max() and L.min() >= 10 and L.max() <= 40
    for b in range(cfg.B):
        k = gi.bf16_bits_to_f32(inp["k_cache"][b])
        assert np.isfinite(k[:L[b]]).all() and np.isnan(k[L[b]:]).all()


def test_planted_agreement_rate():
    cfg = gi.CONFIGS["llama70b"]
    inp = gi.make_inputs(cfg, attn=False)
    hits = total = 0
    for b in range(cfg.B):
        ch = gi.children_of(inp["parents"][b])
        am = inp["logits"][b].argmax(axis=1)
        for v in range(cfg.N):
            if ch[v]:
                total += 1
                hits += int(am[v] in {int(inp["draft_tokens"][b, c]) for c in ch[v]})
    assert abs(hits / total - cfg.p_agree) < 0.05
