"""Pins for the oracle's KV-cache commit: it is a gather of whole rows, so every expected value
is written out directly from the definition with numpy indexing (no oracle code is reused)."""
import numpy as np

import gsd_inputs as gi
import oracle


def small_inputs(seed=0, B=3, Lmax=20, N=9, Hkv=2, D=8, Tcap=6):
    rng = np.random.default_rng(seed)
    kc = rng.integers(0, 2 ** 16, size=(B, Lmax, Hkv, D), dtype=np.uint16)
    vc = rng.integers(0, 2 ** 16, size=(B, Lmax, Hkv, D), dtype=np.uint16)
    dk = rng.integers(0, 2 ** 16, size=(B, N, Hkv, D), dtype=np.uint16)
    dv = rng.integers(0, 2 ** 16, size=(B, N, Hkv, D), dtype=np.uint16)
    return kc, vc, dk, dv


def test_rows_land_behind_the_old_end_and_nothing_else_moves():
    kc, vc, dk, dv = small_inputs()
    nodes = np.array([[0, 2, 5, -1, -1, -1], [0, -1, -1, -1, -1, -1], [0, 1, 3, 4, 8, -1]], dtype=np.int32)
    lens = np.array([3, 1, 5], dtype=np.int32)
    sl = np.array([4, 0, 15], dtype=np.int32)
    k2, v2, sl2, over = oracle.commit_kv(kc, vc, dk, dv, nodes, lens, sl)
    assert over == 0 and list(sl2) == [7, 1, 20]
    want_k, want_v = kc.copy(), vc.copy()
    for b in range(3):
        for i in range(lens[b]):
            want_k[b, sl[b] + i] = dk[b, nodes[b, i]]
            want_v[b, sl[b] + i] = dv[b, nodes[b, i]]
    assert np.array_equal(k2, want_k) and np.array_equal(v2, want_v)
    # the inputs themselves were not modified
    assert not np.array_equal(k2, kc)


def test_overflow_drops_rows_and_clamps_the_length():
    kc, vc, dk, dv = small_inputs(1)
    nodes = np.array([[0, 1, 2, 3, -1, -1]] * 3, dtype=np.int32)
    lens = np.array([4, 4, 4], dtype=np.int32)
    sl = np.array([18, 20, 3], dtype=np.int32)           # room for 2, 0 and 4 rows
    k2, v2, sl2, over = oracle.commit_kv(kc, vc, dk, dv, nodes, lens, sl)
    assert over == 2 and list(sl2) == [20, 20, 7]
    assert np.array_equal(k2[0, 18], dk[0, 0]) and np.array_equal(k2[0, 19], dk[0, 1])
    assert np.array_equal(k2[1], kc[1]) and np.array_equal(v2[1], vc[1])
    assert np.array_equal(v2[2, 3:7], dv[2, :4])


def test_commit_then_attention_equals_attention_over_the_longer_prefix():
    # after the commit, the accepted nodes are ordinary cache rows: a fresh root that sees only
    # itself must attend to exactly the old prefix plus the committed path
    cfg = gi.VerifyConfig("t", 9, 2, 4, 2, 16, (5, 9), 12, 4, 3, 2, 32, 32, 0.9)
    inp = gi.make_inputs(cfg, 3, pad_fill="zero")
    Lmax_old = inp["Lmax"]
    grow = cfg.depth + 1
    kc = np.concatenate([inp["k_cache"], np.zeros((cfg.B, grow, cfg.Hkv, cfg.D), np.uint16)], axis=1)
    vc = np.concatenate([inp["v_cache"], np.zeros((cfg.B, grow, cfg.Hkv, cfg.D), np.uint16)], axis=1)
    _, lens, nodes, _ = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    k2, v2, sl2, over = oracle.commit_kv(kc, vc, inp["draft_k"], inp["draft_v"], nodes, lens, inp["seq_lens"])
    assert over == 0 and np.array_equal(sl2, inp["seq_lens"] + lens) and k2.shape[1] == Lmax_old + grow
    # reference: the old prefix, and the accepted path visible through the mask instead
    mask = np.zeros_like(inp["ancestor_mask"])
    for b in range(cfg.B):
        for v in nodes[b, :lens[b]]:
            mask[b, :, v // 32] |= np.uint32(1 << (v % 32))
    a = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"], mask, inp["seq_lens"])
    b_ = oracle.attn(inp["q"], k2, v2, inp["draft_k"], inp["draft_v"], np.zeros_like(mask), sl2)
    assert np.allclose(a, b_, rtol=0, atol=1e-12)
