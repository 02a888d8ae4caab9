"""Pins for the CPU oracle's attention: closed forms, library attention on the special
cases the paper's rule reduces to, and invariants.  None of these re-uses oracle code."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import gsd_inputs as gi
import oracle
from helpers import mask_bits


def bits(x):
    return gi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(bits_arr):
    return torch.from_numpy(gi.bf16_bits_to_f32(bits_arr).astype(np.float64))


def small_cfg(**kw):
    base = dict(name="t", config_id=9, B=2, Hq=4, Hkv=2, D=16, L=(5, 30), N=40, depth=8,
                kmax=3, pmax=2, V=64, vtok=64, p_agree=0.5)
    base.update(kw)
    return gi.VerifyConfig(**base)


def run_oracle(inp, **kw):
    return oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                       inp["ancestor_mask"], inp["seq_lens"], **kw)


def sdpa_with_mask(inp, b, visible_draft):
    """Library attention (fp64, CPU) for sequence b.  visible_draft[n] lists the draft nodes
    row n may see; all rows see the first seq_lens[b] cache rows.  q-head h uses kv-head
    h // G (contiguous groups, the LLaMA repeat_kv convention)."""
    cfg = inp["cfg"]
    L = int(inp["seq_lens"][b])
    k = torch.cat([f64(inp["k_cache"][b, :L]), f64(inp["draft_k"][b])])   # [L+N, Hkv, D]
    v = torch.cat([f64(inp["v_cache"][b, :L]), f64(inp["draft_v"][b])])
    k = k.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)                # [Hq, L+N, D]
    v = v.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
    q = f64(inp["q"][b]).permute(1, 0, 2)                                  # [Hq, N, D]
    m = torch.zeros(cfg.N, L + cfg.N, dtype=torch.bool)
    m[:, :L] = True
    for n, vis in enumerate(visible_draft):
        for j in vis:
            m[n, L + j] = True
    out = F.scaled_dot_product_attention(q[None], k[None], v[None], attn_mask=m[None, None])
    return out[0].permute(1, 0, 2).numpy()                                 # [N, Hq, D]


# ---------------------------------------------------------------- closed forms
def test_two_key_closed_form_and_scale():
    # one cache key, one draft key (the node itself): out = w*v0 + (1-w)*v1,
    # w = 1 / (1 + exp(s1 - s0)), s = <q,k> / sqrt(D)
    q = bits([[[[1, 2, 0, -1]]]])
    k0 = bits([[[[0.5, 0.5, 1, 1]]]]); v0 = bits([[[[1, 0, 2, 4]]]])
    k1 = bits([[[[1, 0, 0, 0]]]]); v1 = bits([[[[3, 1, 0, -4]]]])
    mask = np.array([[[1]]], dtype=np.uint32)
    out = oracle.attn(q, k0, v0, k1, v1, mask, np.array([1], dtype=np.int32))
    s0, s1 = 0.5 * 0.5, 0.5 * 1.0
    w = 1.0 / (1.0 + math.exp(s1 - s0))
    want = w * np.array([1, 0, 2, 4.0]) + (1 - w) * np.array([3, 1, 0, -4.0])
    assert np.allclose(out[0, 0, 0], want, rtol=0, atol=1e-14)
    out = oracle.attn(q, k0, v0, k1, v1, mask, np.array([1], dtype=np.int32), scale=2.0)
    w = 1.0 / (1.0 + math.exp(2.0 * 1.0 - 2.0 * 0.5))
    want = w * np.array([1, 0, 2, 4.0]) + (1 - w) * np.array([3, 1, 0, -4.0])
    assert np.allclose(out[0, 0, 0], want, rtol=0, atol=1e-14)
    # scores of 1000 and 2000: the row maximum must be subtracted before exponentiating
    out = oracle.attn(q, k0, v0, k1, v1, mask, np.array([1], dtype=np.int32), scale=2000.0)
    assert np.array_equal(out[0, 0, 0], np.array([3, 1, 0, -4.0]))


def test_visibility_probe_uniform_softmax():
    # q = 0 makes the softmax uniform: the output is the plain mean of the visible value
    # rows.  Values encode (key id, 1, kv head, (7*id) % 13), so the means read back which
    # keys were visible: pins seq_lens, bit/word order of the mask and the GQA head mapping.
    cfg = small_cfg()
    inp = gi.make_inputs(cfg, 3, accept=False, pad_fill="nan")
    B, N, Hkv, D, Lmax = cfg.B, cfg.N, cfg.Hkv, cfg.D, inp["Lmax"]
    inp["q"][:] = 0
    vc = np.zeros((B, Lmax, Hkv, D), dtype=np.float32)
    dv = np.zeros((B, N, Hkv, D), dtype=np.float32)
    for c in range(Hkv):
        for j in range(Lmax):
            vc[:, j, c, :4] = [j, 1, c, (7 * j) % 13]
        for j in range(N):
            kid = 100 + j                      # draft ids 100.. (all < 256: exact in bf16)
            dv[:, j, c, :4] = [kid, 1, c, (7 * kid) % 13]
    inp["v_cache"] = gi.f32_to_bf16_bits(vc)
    inp["draft_v"] = gi.f32_to_bf16_bits(dv)
    out = run_oracle(inp)
    for b in range(B):
        L = int(inp["seq_lens"][b])
        for n in range(N):
            ids = list(range(L)) + [100 + j for j in mask_bits(inp["ancestor_mask"][b, n], N)]
            for h in range(cfg.Hq):
                want = [np.mean(ids), 1.0, h // cfg.G, np.mean([(7 * i) % 13 for i in ids])]
                assert np.allclose(out[b, n, h, :4], want, rtol=0, atol=1e-12)
                assert np.all(out[b, n, h, 4:] == 0)


def test_dominant_key_selects_its_value_row():
    cfg = small_cfg(B=1, Hq=2, Hkv=2, L=20, N=8, depth=3)
    inp = gi.make_inputs(cfg, 5, accept=False)
    # make cache key 7 of kv-head 1 align with every query of head 1 with a huge score
    qf = gi.bf16_bits_to_f32(inp["q"])
    qf[0, :, 1, :] = 0
    qf[0, :, 1, 3] = 16.0
    kf = gi.bf16_bits_to_f32(inp["k_cache"])
    kf[0, :, 1, 3] = 0
    kf[0, 7, 1, 3] = 16.0           # score 256/4 = 64 above the others
    inp["q"], inp["k_cache"] = gi.f32_to_bf16_bits(qf), gi.f32_to_bf16_bits(kf)
    dk = gi.bf16_bits_to_f32(inp["draft_k"]); dk[0, :, 1, 3] = 0
    inp["draft_k"] = gi.f32_to_bf16_bits(dk)
    out = run_oracle(inp)
    want = gi.bf16_bits_to_f32(inp["v_cache"])[0, 7, 1].astype(np.float64)
    assert np.allclose(out[0, :, 1, :], want[None], atol=1e-20 + 1e-24, rtol=1e-12)


# ---------------------------------------------------------------- library special cases
def test_chain_dag_is_causal_attention():
    # a chain 0->1->...->N-1 gives a lower-triangular mask: ordinary causal attention over
    # the concatenation [prefix; draft] (sequence-structured drafting, Sec. 3)
    cfg = small_cfg(N=37, depth=36, kmax=1, pmax=1)
    inp = gi.make_inputs(cfg, 11, accept=False, pad_fill="nan")
    assert all(inp["parents"][0][v] == [v - 1] for v in range(1, cfg.N))
    out = run_oracle(inp)
    for b in range(cfg.B):
        L = int(inp["seq_lens"][b])
        k = torch.cat([f64(inp["k_cache"][b, :L]), f64(inp["draft_k"][b])])
        v = torch.cat([f64(inp["v_cache"][b, :L]), f64(inp["draft_v"][b])])
        k = k.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        v = v.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        # full causal self-attention over L+N positions; the draft rows are the last N.
        # Queries of the prefix positions are irrelevant for those rows.
        qfull = torch.zeros(cfg.Hq, L + cfg.N, cfg.D, dtype=torch.float64)
        qfull[:, L:] = f64(inp["q"][b]).permute(1, 0, 2)
        ref = F.scaled_dot_product_attention(qfull[None], k[None], v[None], is_causal=True)
        ref = ref[0, :, L:].permute(1, 0, 2).numpy()
        assert np.allclose(out[b], ref, rtol=0, atol=1e-12)


def test_tree_dag_is_per_path_sequential_decoding():
    # in a tree every node has one root path; its row equals ordinary causal attention of
    # that path appended to the prefix (tree attention, Sec. 4.1)
    cfg = small_cfg(B=1, N=30, depth=5, kmax=3, pmax=1, L=17)
    inp = gi.make_inputs(cfg, 13, accept=False)
    parents = inp["parents"][0]
    out = run_oracle(inp)
    L = cfg.L
    checked = 0
    for leaf in range(cfg.N):
        path = [leaf]
        while parents[path[-1]]:
            path.append(parents[path[-1]][0])
        path = path[::-1]
        idx = torch.tensor(path)
        k = torch.cat([f64(inp["k_cache"][0, :L]), f64(inp["draft_k"][0])[idx]])
        v = torch.cat([f64(inp["v_cache"][0, :L]), f64(inp["draft_v"][0])[idx]])
        k = k.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        v = v.repeat_interleave(cfg.G, dim=1).permute(1, 0, 2)
        qfull = torch.zeros(cfg.Hq, L + len(path), cfg.D, dtype=torch.float64)
        qfull[:, L:] = f64(inp["q"][0])[idx].permute(1, 0, 2)
        ref = F.scaled_dot_product_attention(qfull[None], k[None], v[None], is_causal=True)
        ref = ref[0, :, L:].permute(1, 0, 2).numpy()          # [len(path), Hq, D]
        assert np.allclose(out[0, path], ref, rtol=0, atol=1e-12)
        checked += 1
    assert checked == cfg.N


def test_all_bits_set_is_unmasked_attention():
    cfg = small_cfg()
    inp = gi.make_inputs(cfg, 17, accept=False, pad_fill="nan")
    inp["ancestor_mask"][:] = 0xFFFFFFFF        # including the padding bits >= N
    out = run_oracle(inp)
    for b in range(cfg.B):
        ref = sdpa_with_mask(inp, b, [range(cfg.N)] * cfg.N)
        assert np.allclose(out[b], ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("name", ["tiny", "dag40"])
def test_general_dag_mask_against_library_attention(name):
    cfg = gi.CONFIGS["tiny"] if name == "tiny" else small_cfg(pmax=3)
    inp = gi.make_inputs(cfg, 19, accept=False, pad_fill="nan")
    assert any(len(p) > 1 for ps in inp["parents"] for p in ps)    # really a DAG
    out = run_oracle(inp)
    for b in range(cfg.B):
        vis = [mask_bits(inp["ancestor_mask"][b, n], cfg.N) for n in range(cfg.N)]
        ref = sdpa_with_mask(inp, b, vis)
        assert np.allclose(out[b], ref, rtol=0, atol=1e-12)


def test_arbitrary_bit_patterns_are_honoured_literally():
    # not lower-triangular, no diagonal: the mask is data, nothing is added implicitly
    cfg = small_cfg(B=1, L=9)
    inp = gi.make_inputs(cfg, 23, accept=False)
    rng = np.random.default_rng(1)
    inp["ancestor_mask"] = rng.integers(0, 2 ** 32, size=inp["ancestor_mask"].shape,
                                        dtype=np.uint32)
    out = run_oracle(inp)
    vis = [mask_bits(inp["ancestor_mask"][0, n], cfg.N) for n in range(cfg.N)]
    ref = sdpa_with_mask(inp, 0, vis)
    assert np.allclose(out[0], ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- invariants, edge cases
def test_prefix_permutation_invariance():
    cfg = small_cfg(B=1, L=25)
    inp = gi.make_inputs(cfg, 29, accept=False)
    a = run_oracle(inp)
    perm = np.random.default_rng(2).permutation(cfg.L)
    inp["k_cache"] = np.ascontiguousarray(inp["k_cache"][:, perm])
    inp["v_cache"] = np.ascontiguousarray(inp["v_cache"][:, perm])
    assert np.allclose(a, run_oracle(inp), rtol=0, atol=1e-12)


def test_padding_rows_are_invisible():
    cfg = small_cfg()
    a = run_oracle(gi.make_inputs(cfg, 31, accept=False, pad_fill="nan"))
    b = run_oracle(gi.make_inputs(cfg, 31, accept=False, pad_fill="junk"))
    assert np.isfinite(a).all() and np.array_equal(a, b)


def test_empty_key_set_gives_zeros_and_self_only_gives_own_value():
    cfg = small_cfg(B=1, L=0, N=8, depth=3)
    inp = gi.make_inputs(cfg, 37, accept=False)
    assert inp["k_cache"].shape[1] == 1            # a dummy row that must stay invisible
    inp["ancestor_mask"][:] = 0
    inp["ancestor_mask"][0, 3, 0] = 1 << 3         # node 3 sees itself only
    out = run_oracle(inp)
    dv = gi.bf16_bits_to_f32(inp["draft_v"]).astype(np.float64)
    for n in range(cfg.N):
        for h in range(cfg.Hq):
            want = dv[0, 3, h // cfg.G] if n == 3 else np.zeros(cfg.D)
            assert np.array_equal(out[0, n, h], want)


def test_row_subset_matches_full():
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, accept=False)
    full = run_oracle(inp)
    rows = [(0, 0, 0), (0, 15, 3), (0, 7, 2)]
    sub = oracle.attn_rows(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"],
                           inp["draft_v"], inp["ancestor_mask"], inp["seq_lens"], rows)
    for i, (b, n, h) in enumerate(rows):
        assert np.array_equal(sub[i], full[b, n, h])
