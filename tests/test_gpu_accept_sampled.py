"""gsd_accept_sampled on the GPU against the CPU oracle.  The kernel accumulates the softmax
statistics in fp32, the oracle in fp64; a decision "u q < p" or "cumulative sum > u" is an
integer taken from floating point, so the random numbers of these tests are placed at least 2 %
(relative) away from every threshold they are compared with.  With that the results are unique
and compared bit by bit."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors

pytestmark = pytest.mark.gpu


def softmax64(x):
    x = x.astype(np.float64)
    m = np.max(x, axis=-1, keepdims=True)
    e = np.exp(x - m)
    return e / e.sum(axis=-1, keepdims=True)


def decisive_inputs(inp, seed, q_lo=0.5, q_hi=6.0):
    """draft_q, u_accept, u_sample with a margin from every threshold; returns them and the oracle's answer."""
    rng = np.random.default_rng(seed)
    lg, tok, ptr, idx = inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"]
    B, N, V = lg.shape
    q = np.ones((B, N), dtype=np.float32)
    u = np.zeros((B, N), dtype=np.float32)
    for b in range(B):
        P = softmax64(lg[b])
        for v in range(1, N):
            probs = np.array([P[p, tok[b, v]] for p in idx[b, ptr[b, v]:ptr[b, v + 1]]])
            ref = float(probs.max()) if len(probs) else 0.5
            # a draft probability around the target's, so that both outcomes occur
            q[b, v] = np.float32(min(1.0, max(1e-6, ref * rng.uniform(q_lo, q_hi))))
            for _ in range(100):
                cand = np.float32(rng.uniform(0, 1))
                prod = float(cand) * float(q[b, v])
                if all(abs(prod - p) > 0.02 * max(p, 1e-30) for p in probs):
                    u[b, v] = cand
                    break
            else:
                u[b, v] = 0.0
    us = np.full((B,), 0.5, dtype=np.float32)
    _, lens, nodes = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us)
    for b in range(B):
        end = nodes[b, lens[b] - 1]
        P = softmax64(lg[b, end])
        cdf = np.cumsum(P)
        heavy = np.flatnonzero(P > 1e-4)
        t = int(rng.choice(heavy))
        lo = cdf[t] - P[t]
        us[b] = np.float32(lo + P[t] * rng.uniform(0.25, 0.75))      # well inside the token's interval
    want = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us)
    return q, u, us, want


def run_gpu(inp, q, u, us, status=None):
    import paper_2407_16207_b200 as gsd
    t = accept_tensors(inp)
    dev = t["logits"].device
    toks, lens, nodes = gsd.gsd_accept_sampled(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"],
                                               torch.from_numpy(q).to(dev), torch.from_numpy(u).to(dev),
                                               torch.from_numpy(us).to(dev), status=status)
    torch.cuda.synchronize()
    return toks.cpu().numpy(), lens.cpu().numpy(), nodes.cpu().numpy()


def check(inp, seed, **kw):
    q, u, us, want = decisive_inputs(inp, seed, **kw)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = run_gpu(inp, q, u, us, status=status)
    assert int(status.item()) == 0
    assert np.array_equal(got[1], want[1])
    assert np.array_equal(got[0], want[0])
    assert np.array_equal(got[2], want[2])
    return want


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
@pytest.mark.parametrize("trial", [0, 1])
def test_configs_bit_exact(name, trial):
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False)
    want = check(inp, 100 + trial)
    if name != "tiny":
        assert want[1].max() > 1 and want[1].min() < inp["logits"].shape[1]   # both outcomes occur


def test_everything_accepted_and_everything_rejected():
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, attn=False)
    B, N = cfg.B, cfg.N
    q = np.ones((B, N), dtype=np.float32)
    us = np.full((B,), 0.5, dtype=np.float32)
    lens = {}
    for u_val in (0.0, 0.99999):
        # u q = 0.99999 is above every probability of these logits; 0 is below every one
        u = np.full((B, N), u_val, dtype=np.float32)
        want = oracle.accept_sampled(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u, us)
        got = run_gpu(inp, q, u, us)
        assert np.array_equal(got[1], want[1]) and np.array_equal(got[2], want[2])
        lens[u_val] = want[1]
    assert (lens[0.99999] == 1).all()
    assert all(lens[0.0][b] == max(inp["levels"][b]) + 1 for b in range(B))


def test_vocabulary_not_a_multiple_of_four_and_filtered_entries():
    # scalar load path; entries at -inf (nucleus filtering) carry no mass and are never drawn
    cfg = gi.VerifyConfig("t", 7, 3, 8, 1, 128, 64, 48, 8, 4, 3, 1003, 1003, 0.6)
    inp = gi.make_inputs(cfg, 11, attn=False)
    lg = inp["logits"].copy()
    rng = np.random.default_rng(3)
    drop = rng.uniform(size=lg.shape) < 0.5
    am = oracle.argmax(lg)
    np.put_along_axis(drop, am[..., None].astype(np.int64), False, axis=-1)   # keep one finite entry per row
    lg[drop] = -np.inf
    inp["logits"] = lg
    check(inp, 7)


def test_one_hot_targets_give_the_deterministic_result():
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["llama13b"]
    inp = gi.make_inputs(cfg, attn=False)
    am = oracle.argmax(inp["logits"])
    lg = np.full(inp["logits"].shape, -80.0, dtype=np.float32)
    np.put_along_axis(lg, am[..., None].astype(np.int64), 0.0, axis=-1)
    inp["logits"] = lg
    rng = np.random.default_rng(2)
    q = np.ones((cfg.B, cfg.N), dtype=np.float32)
    u = rng.uniform(0.01, 0.99, size=(cfg.B, cfg.N)).astype(np.float32)
    us = rng.uniform(0.01, 0.99, size=(cfg.B,)).astype(np.float32)
    got = run_gpu(inp, q, u, us)
    t = accept_tensors(inp)
    toks, lens, nodes = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
    assert np.array_equal(got[0], toks.cpu().numpy()) and np.array_equal(got[1], lens.cpu().numpy())
    assert np.array_equal(got[2], nodes.cpu().numpy())


def test_row_without_mass_is_flagged_and_repeat_calls_agree():
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, attn=False)
    q, u, us, want = decisive_inputs(inp, 5)
    a = run_gpu(inp, q, u, us)
    b = run_gpu(inp, q, u, us)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    bad = dict(inp)
    lg = inp["logits"].copy()
    lg[0, 1, :] = -np.inf
    bad["logits"] = lg
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    run_gpu(bad, q, u, us, status=status)
    assert int(status.item()) & 0x40
