"""gsd_accept_sampled on the GPU against the CPU oracle.  The kernel accumulates the softmax
statistics in fp32, the oracle in fp64; a decision "u q < p" or "cumulative weight > u" is an
integer taken from floating point.  `test_measured_error_of_the_probabilities` measures how far
the kernel's probabilities and cumulative weights are from fp64 (by bisection on the random
numbers); the other tests keep their random numbers MARGIN_P (relative) away from every
probability and MARGIN_CDF (absolute, in units of the total weight) away from every boundary of
the cumulative distribution, a few times the measured error.  With that the results are unique
and compared bit by bit."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors

pytestmark = pytest.mark.gpu

MARGIN_P = 1e-4      # relative distance of u q from every target probability it is compared with
MARGIN_CDF = 1e-4    # distance of u_sample from the ends of the chosen token's interval


def softmax64(x):
    x = x.astype(np.float64)
    m = np.max(x, axis=-1, keepdims=True)
    e = np.exp(x - m)
    return e / e.sum(axis=-1, keepdims=True)


def draft_logits_for(lg, seed, noise=0.7):
    """Draft-model logits: the target's plus noise, so that P and Q resemble each other."""
    rng = np.random.default_rng(seed)
    return (lg + noise * rng.standard_normal(lg.shape).astype(np.float32)).astype(np.float32)


def regeneration_weights(lg_row, dl_row, has_child):
    """The weights the regenerated token is drawn from, in the test's own terms (numpy fp64)."""
    P = softmax64(lg_row)
    if dl_row is not None and has_child:
        r = np.maximum(P - softmax64(dl_row), 0.0)
        if r.sum() > 1e-6:
            return r / r.sum()
    return P


def decisive_inputs(inp, seed, q_lo=0.5, q_hi=6.0, dl=None):
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
                if all(abs(prod - p) > MARGIN_P * max(p, 1e-30) for p in probs):
                    u[b, v] = cand
                    break
            else:
                u[b, v] = 0.0
    us = np.full((B,), 0.5, dtype=np.float32)
    _, lens, nodes = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us, draft_logits=dl)
    for b in range(B):
        end = nodes[b, lens[b] - 1]
        has_child = bool((idx[b, :ptr[b, N]] == end).any())
        w = regeneration_weights(lg[b, end], None if dl is None else dl[b, end], has_child)
        cdf = np.cumsum(w)
        heavy = np.flatnonzero(w > 10 * MARGIN_CDF)
        t = int(rng.choice(heavy)) if len(heavy) else int(np.argmax(w))
        margin = min(MARGIN_CDF, 0.25 * w[t])       # a flat row has no token 10 margins wide
        lo = cdf[t] - w[t]
        us[b] = np.float32(rng.uniform(lo + margin, cdf[t] - margin))   # inside the token's interval
        assert lo + 0.5 * margin < float(us[b]) < cdf[t] - 0.5 * margin
    want = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us, draft_logits=dl)
    return q, u, us, want


def run_gpu(inp, q, u, us, status=None, dl=None):
    import paper_2407_16207_b200 as gsd
    t = accept_tensors(inp)
    dev = t["logits"].device
    toks, lens, nodes = gsd.gsd_accept_sampled(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"],
                                               torch.from_numpy(q).to(dev), torch.from_numpy(u).to(dev),
                                               torch.from_numpy(us).to(dev), status=status,
                                               draft_logits=None if dl is None else torch.from_numpy(dl).to(dev))
    torch.cuda.synchronize()
    return toks.cpu().numpy(), lens.cpu().numpy(), nodes.cpu().numpy()


def check(inp, seed, dl=None, **kw):
    q, u, us, want = decisive_inputs(inp, seed, dl=dl, **kw)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = run_gpu(inp, q, u, us, status=status, dl=dl)
    assert int(status.item()) == 0
    assert np.array_equal(got[1], want[1])
    assert np.array_equal(got[0], want[0])
    assert np.array_equal(got[2], want[2])
    return want


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
@pytest.mark.parametrize("trial", [0, 1])
def test_configs_bit_exact_with_residual(name, trial):
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False)
    dl = draft_logits_for(inp["logits"], 300 + trial)
    want = check(inp, 200 + trial, dl=dl)
    if cfg.B > 1:
        # the residual really is what decided some of the tokens: some hypothesis ends at a node
        # with (rejected) children, and there the drawn token has more target than draft mass
        used = 0
        for b in range(cfg.B):
            end = want[2][b, want[1][b] - 1]
            if (inp["parent_idx"][b, :inp["parent_ptr"][b, cfg.N]] == end).any():
                t = want[0][b, want[1][b] - 1]
                assert softmax64(inp["logits"][b, end])[t] > softmax64(dl[b, end])[t]
                used += 1
        assert used > 0


def test_residual_special_cases():
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, attn=False)
    B, N = cfg.B, cfg.N
    lg = inp["logits"]
    q = np.ones((B, N), dtype=np.float32)
    # (1) every step rejected, draft distribution == target distribution: no residual mass, P is used
    u = np.full((B, N), 0.99999, dtype=np.float32)
    us = np.full((B,), 0.5, dtype=np.float32)
    w = softmax64(lg[0, 0]); cdf = np.cumsum(w); t = int(np.argmax(w))
    us[0] = np.float32(cdf[t] - 0.5 * w[t])       # the middle of the root's heaviest token
    want = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u, us, draft_logits=lg)
    assert want[1][0] == 1 and want[0][0, 0] == t
    plain = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u, us)
    assert np.array_equal(want[0], plain[0])
    got = run_gpu(inp, q, u, us, dl=lg.copy())
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    # (2) every step accepted: the end node is a leaf, P is used whatever the draft logits are
    u0 = np.zeros((B, N), dtype=np.float32)
    dl = draft_logits_for(lg, 9)
    want = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u0, us, draft_logits=dl)
    plain = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u0, us)
    assert np.array_equal(want[0], plain[0])
    # u_sample = 0.5 may sit on a boundary: place it with the margin first
    end = want[2][0, want[1][0] - 1]
    w = softmax64(lg[0, end]); cdf = np.cumsum(w); t = int(np.argmax(w))
    us[0] = np.float32(cdf[t] - 0.5 * w[t])
    want = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u0, us, draft_logits=dl)
    got = run_gpu(inp, q, u0, us, dl=dl)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
    # (3) a draft row without mass is flagged
    bad = dl.copy(); bad[0, 0, :] = -np.inf
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    run_gpu(inp, q, u, us, status=status, dl=bad)
    assert int(status.item()) & 0x40


def test_measured_error_of_the_probabilities():
    """How far are the kernel's fp32 probabilities from fp64?  512 two-node chains with random
    rows (V = 32000); the flip point of the step's test in u (with q = 1) IS the kernel's
    probability of the child's token, found by bisection over 26 calls; likewise the flip point of
    the regenerated token in u_sample is the kernel's cumulative weight below that token.  The
    margins used by the other tests in this file are >= 10 times what is measured here."""
    B, N, V = 512, 2, 32000
    rng = np.random.default_rng(77)
    lg = rng.standard_normal((B, N, V)).astype(np.float32)
    tok = np.zeros((B, N), dtype=np.int32)
    tok[:, 1] = rng.integers(0, V, size=B)
    # some heavy tokens, so that probabilities span 3e-5 .. 0.5
    lg[np.arange(B), 0, tok[:, 1]] += rng.uniform(0, 10, size=B).astype(np.float32)
    ptr = np.tile(np.array([0, 0, 1], dtype=np.int32), (B, 1))
    idx = np.zeros((B, 1), dtype=np.int32)
    inp = dict(logits=lg, draft_tokens=tok, parent_ptr=ptr, parent_idx=idx)
    P = softmax64(lg[:, 0])
    p_true = P[np.arange(B), tok[:, 1]]
    q = np.ones((B, N), dtype=np.float32)
    us = np.full((B,), 0.5, dtype=np.float32)
    lo = np.zeros(B); hi = np.ones(B)
    for _ in range(26):
        mid = (0.5 * (lo + hi)).astype(np.float32)
        u = np.zeros((B, N), dtype=np.float32); u[:, 1] = mid
        _, lens, _ = run_gpu(inp, q, u, us)
        acc = lens == 2
        lo = np.where(acc, mid, lo); hi = np.where(acc, hi, mid)
    rel = np.abs(0.5 * (lo + hi) - p_true) / p_true
    # the bisection itself resolves one float32 step of u (6e-8 absolute)
    rel_floor = 1.2e-7 / p_true
    big = p_true > 1e-2
    print(f"probability: max relative error {np.max(rel[big]):.2e} over the {big.sum()} steps with p > 0.01 "
          f"(median over all {np.median(rel):.2e})")
    assert np.all(rel < 1e-5 + rel_floor)
    # cumulative weights of the residual at the root: every step rejected (u = 0.99999 with q = 1)
    dl = draft_logits_for(lg, 5)
    u = np.full((B, N), 0.99999, dtype=np.float32)
    w = np.stack([regeneration_weights(lg[b, 0], dl[b, 0], True) for b in range(B)])
    cdf = np.cumsum(w, axis=1)
    t = np.array([rng.choice(np.flatnonzero(w[b] > 1e-3)) for b in range(B)])
    edge = cdf[np.arange(B), t] - w[np.arange(B), t]       # cumulative weight below token t
    lo = np.maximum(edge - 5e-4, 0.0); hi = edge + 5e-4
    for _ in range(16):
        mid = (0.5 * (lo + hi)).astype(np.float32)
        toks, lens, _ = run_gpu(inp, q, u, mid, dl=dl)
        assert (lens == 1).all()
        below = toks[:, 0] < t
        assert np.all(toks[:, 0] <= t)
        lo = np.where(below, mid, lo); hi = np.where(below, hi, mid)
    err = np.abs(0.5 * (lo + hi) - edge)
    print(f"cumulative residual weight: max absolute error {np.max(err):.2e} (median {np.median(err):.2e})")
    assert np.all(err < 1e-5)


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


def test_more_rows_than_one_launch_holds():
    # B * N = 70400 rows go out as two launches of whole sequences
    cfg = gi.VerifyConfig("many", 6, 1100, 1, 1, 64, 8, 64, 8, 3, 2, 128, 128, 0.7)
    inp = gi.make_inputs(cfg, attn=False)
    dl = draft_logits_for(inp["logits"], 17)
    check(inp, 31, dl=dl)


def test_row_pointers_that_go_backwards_are_flagged_and_made_safe():
    # the same sanitising rule as gsd_accept (running maximum from zero, bad parents ignored);
    # with every u = 0 each surviving step is accepted
    from test_gpu_accept import sanitised_parents
    N, Ecap, V = 6, 8, 16
    ptr = [0, 0, 1, 5, 3, 4, 6]
    idx = np.array([[0, 0, 1, 1, 2, 3, 4, 2]], dtype=np.int32)
    rng = np.random.default_rng(3)
    inp = dict(logits=rng.standard_normal((1, N, V)).astype(np.float32),
               draft_tokens=rng.integers(0, V, size=(1, N)).astype(np.int32),
               parent_ptr=np.array([ptr], dtype=np.int32), parent_idx=idx)
    q = np.ones((1, N), dtype=np.float32)
    u = np.zeros((1, N), dtype=np.float32)
    end_w = None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    parents = sanitised_parents(ptr, idx[0], N)
    cptr, cidx = gi.parents_to_csr([parents], Ecap)
    us = np.array([0.5], dtype=np.float32)
    _, lens, nodes = oracle.accept_sampled(inp["logits"], inp["draft_tokens"], cptr, cidx, q, u, us)
    w = softmax64(inp["logits"][0, nodes[0, lens[0] - 1]]); t = int(np.argmax(w))
    us[0] = np.float32(np.cumsum(w)[t] - 0.5 * w[t])
    want = oracle.accept_sampled(inp["logits"], inp["draft_tokens"], cptr, cidx, q, u, us)
    got = run_gpu(inp, q, u, us, status=status)
    assert int(status.item()) & 0x1
    for g, w_ in zip(got, want):
        assert np.array_equal(g, w_)
