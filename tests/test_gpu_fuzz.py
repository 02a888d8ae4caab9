"""Seeded random shapes, graphs, vocabularies, kernels and plans against the oracle: a broad sweep
beside the hand-picked cases of the other files (a few hundred cases, some tens of seconds)."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
import test_gpu_accept_sampled as sampled_cases
import test_gpu_draft as draft_cases
from gpu_util import accept_tensors, attn_tensors, out_to_f64

pytestmark = pytest.mark.gpu


def depth_for(N, rng, extra=4):
    # deep enough for N nodes with out-degree 3
    return 0 if N == 1 else int(np.ceil(np.log(2 * N + 1) / np.log(3))) + int(rng.integers(0, extra))


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_attention_random_shapes_kernels_and_plans(seed):
    import paper_2407_16207_b200 as gsd
    rng = np.random.default_rng(seed)
    ran = 0
    for _ in range(40):
        G = int(rng.choice([1, 2, 4, 8, 16]))
        Hkv = int(rng.choice([1, 2, 3, 4]))
        D = int(rng.choice([128, 128, 128, 64]))
        B = int(rng.integers(1, 7))
        N = int(rng.choice([1, 2, 7, 16, 31, 32, 33, 64, 65, 100, 128, 129, 200, 256, 300]))
        lo = int(rng.choice([0, 0, 1, 50, 128]))
        hi = max(lo, int(rng.choice([lo, lo + 1, 127, 128, 129, 260, 500, 900])))
        cfg = gi.VerifyConfig("f", 7, B, Hkv * G, Hkv, D, (lo, hi) if hi > lo else lo, N, depth_for(N, rng), 3, 2, 8, 8, 0.5)
        inp = gi.make_inputs(cfg, int(rng.integers(1, 1 << 30)), accept=False, pad_fill="nan")
        if rng.uniform() < 0.2:      # arbitrary mask bits instead of ancestor sets
            inp["ancestor_mask"] = rng.integers(0, 2 ** 32, size=inp["ancestor_mask"].shape, dtype=np.uint32)
        want = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                           inp["ancestor_mask"], inp["seq_lens"])
        t = attn_tensors(inp)
        for kernel in (1, 2, 0):
            for ns in (0, int(rng.choice([1, 2, 3, 5])), -1, -2):
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                try:
                    out = gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                                              t["ancestor_mask"], t["seq_lens"], kernel=kernel, num_splits=ns, status=status)
                except gsd.GsdError as e:
                    if e.code == -6:         # the tcgen05 kernel does not take this shape
                        continue
                    raise
                torch.cuda.synchronize()
                got = out_to_f64(out)
                what = (cfg, inp["seed"], kernel, ns)
                assert np.isfinite(got).all(), what
                # (rows that see a handful of keys keep values of a few units: error relative to max(1, |value|))
                err = np.abs(got - want) / np.maximum(1.0, np.abs(want))
                assert err.max() <= 1e-2 and err.mean() <= 1e-3, what
                assert int(status.item()) == 0, what
                ran += 1
    assert ran > 300


@pytest.mark.parametrize("seed", [1, 2])
def test_acceptance_masks_and_trees_on_random_graphs(seed):
    import paper_2407_16207_b200 as gsd
    rng = np.random.default_rng(100 + seed)
    sampled = 0
    for _ in range(80):
        B = int(rng.integers(1, 6))
        N = int(rng.choice([1, 2, 5, 17, 33, 64, 100, 200, 256, 400, 512]))
        V = int(rng.choice([2, 7, 64, 257, 1000, 1003, 4096, 32000]))
        cfg = gi.VerifyConfig("f", 7, B, 1, 1, 64, 8, N, depth_for(N, rng, 5), 3, int(rng.integers(1, 4)), V,
                              min(V, int(rng.choice([2, 8, 64, 32000]))), float(rng.uniform(0.2, 0.95)))
        inp = gi.make_inputs(cfg, int(rng.integers(1, 1 << 30)), attn=False)
        t = accept_tensors(inp)
        what = (cfg, inp["seed"])
        want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        got = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
        for g, w in zip(got, want[:3]):
            assert np.array_equal(g.cpu().numpy(), w), what
        mask = gsd.gsd_build_mask(t["parent_ptr"], t["parent_idx"])
        assert np.array_equal(mask.cpu().numpy().view(np.uint32), inp["ancestor_mask"]), what
        Ucap, max_depth = int(rng.choice([N, 2 * N, 64, 1000])), int(rng.choice([2, 5, 99]))
        want_tree = oracle.unmerge_tree(inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], Ucap, max_depth)
        got_tree = gsd.gsd_unmerge_tree(t["draft_tokens"], t["parent_ptr"], t["parent_idx"], Ucap=Ucap, max_depth=max_depth)
        for g, w in zip(got_tree[:4], want_tree[:4]):
            assert np.array_equal(g.cpu().numpy(), w), what + (Ucap, max_depth)
        if V < 7 or N > 256:
            continue
        for with_draft_logits in (False, True):
            dl = sampled_cases.draft_logits_for(inp["logits"], int(rng.integers(1, 1 << 30))) if with_draft_logits else None
            q, u, us, want_s = sampled_cases.decisive_inputs(inp, int(rng.integers(1, 1 << 30)), dl=dl)
            got_s = sampled_cases.run_gpu(inp, q, u, us, dl=dl)
            for g, w in zip(got_s, want_s[:3]):
                assert np.array_equal(g, w), what + (with_draft_logits,)
            sampled += 1
    assert sampled > 60


@pytest.mark.parametrize("seed", [1, 2])
def test_draft_growth_random_runs(seed):
    rng = np.random.default_rng(200 + seed)
    done = 0
    for _ in range(150):
        V = int(rng.choice([6, 17, 64, 257, 1003, 4096, 32000]))
        k = int(rng.choice([1, 2, 3, 4, 8]))
        if V <= k + 1:
            continue
        draft_cases.grow_levels(B=int(rng.integers(1, 5)), V=V, k=k, tau=int(rng.integers(1, 5)), levels=int(rng.integers(2, 7)),
                                Ncap=int(rng.choice([30, 100, 512])), seed=int(rng.integers(1, 1 << 30)),
                                logit_scale=float(rng.choice([0.5, 1.0, 3.0])),
                                round_to=(float(rng.choice([0.25, 0.5, 1.0])) if rng.uniform() < 0.4 else None),
                                drop=(float(rng.uniform(0.1, 0.9)) if rng.uniform() < 0.3 else 0.0))
        done += 1
    assert done > 100
