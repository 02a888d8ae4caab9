"""Pins of the oracle's non-deterministic verification (Sec. 3: accept with probability
min(1, p/q), the first rejection ends the hypothesis, the target model regenerates that token;
Sec. 6.4: the same on the token graph).  The random numbers are inputs, so every case is exact."""
import numpy as np
import pytest

import gsd_inputs as gi
import oracle

LOG = np.log


def chain(n):
    """parent CSR of the path 0 -> 1 -> ... -> n-1"""
    ptr = np.array([[0] + list(range(0, n))], dtype=np.int32)
    idx = np.array([list(range(0, n - 1)) or [0]], dtype=np.int32)
    return ptr, idx


def run(logits, tok, ptr, idx, q, u, us):
    t, l, nd = oracle.accept_sampled(np.asarray(logits, np.float32)[None], np.asarray(tok, np.int32)[None], ptr, idx,
                                     np.asarray(q, np.float32)[None], np.asarray(u, np.float32)[None],
                                     np.asarray([us], np.float32))
    n = int(l[0])
    return list(t[0, :n]), list(nd[0, :n])


def test_worked_chain():
    # P rows: node 0 -> [.5,.25,.125,.125]; node 1 -> [.1,.2,.3,.4]; tokens of nodes 1..3: 0, 0, 2
    P = np.array([[.5, .25, .125, .125], [.1, .2, .3, .4], [.25, .25, .25, .25], [.7, .1, .1, .1]])
    ptr, idx = chain(4)
    tok = [3, 0, 0, 2]
    # step 0->1: u q = .5*.8 = .4 < .5 accepted; step 1->2: .3*.5 = .15 < .1 is false: rejected
    toks, nodes = run(LOG(P), tok, ptr, idx, q=[1, .8, .5, .5], u=[0, .5, .3, .0], us=0.25)
    assert nodes == [0, 1]
    # regenerated at node 1: cumulative .1, .3 -> the first one above .25 is index 1
    assert toks == [0, 1]
    # with a smaller u the second step passes too (.1*.5 = .05 < .1) and the third (0 < .25)
    toks, nodes = run(LOG(P), tok, ptr, idx, q=[1, .8, .5, .5], u=[0, .5, .1, .0], us=0.95)
    assert nodes == [0, 1, 2, 3]
    assert toks == [0, 0, 2, 3]          # .7+.1+.1 = .9 is not above .95: index 3


def test_strict_comparisons():
    # V = 2 with equal logits: both probabilities are exactly one half
    ptr, idx = chain(2)
    lg = np.zeros((2, 2))
    # u q == p is a rejection; just below is an acceptance
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .5], us=.1)[1] == [0]
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, np.nextafter(np.float32(.5), np.float32(0))], us=.1)[1] == [0, 1]
    # inverse CDF: the cumulative value has to exceed u
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .9], us=.5)[0] == [1]
    assert run(lg, [0, 1], ptr, idx, q=[1, 1], u=[0, .9], us=.49)[0] == [0]


def test_draft_probability_scales_the_test():
    # p = 1/4; with q = 1/8 the ratio is above one: always accepted; with q = 1 only below 1/4
    ptr, idx = chain(2)
    lg = np.zeros((2, 4))
    assert run(lg, [0, 2], ptr, idx, q=[1, .125], u=[0, .999], us=.1)[1] == [0, 1]
    assert run(lg, [0, 2], ptr, idx, q=[1, 1.0], u=[0, .26], us=.1)[1] == [0]
    assert run(lg, [0, 2], ptr, idx, q=[1, 1.0], u=[0, .24], us=.1)[1] == [0, 1]
    # q = 0 (the draft gave the token no mass): accepted whenever the target gives it any
    assert run(lg, [0, 2], ptr, idx, q=[1, 0.0], u=[0, .999], us=.1)[1] == [0, 1]


def test_probability_is_read_from_the_parent_on_the_path():
    # node 3 (token 1) has the parents 1 and 2; node 1 gives token 1 mass .9, node 2 gives .05
    P = np.array([[.5, .5, 0, 0], [.05, .9, .05, 0], [.9, .05, .05, 0], [.25, .25, .25, .25]])
    with np.errstate(divide="ignore"):
        lg = LOG(P)
    ptr = np.array([[0, 0, 1, 2, 4]], dtype=np.int32)
    idx = np.array([[0, 0, 1, 2]], dtype=np.int32)
    tok = [0, 0, 1, 1]
    # u q = .5 for node 3: passes under node 1 only; nodes 1 and 2 both pass under the root
    toks, nodes = run(lg, tok, ptr, idx, q=[1, 1, 1, 1], u=[0, .4, .4, .5], us=.1)
    assert nodes == [0, 1, 3] and toks[:2] == [0, 1]
    # make the step 0 -> 1 fail: the only way to node 3 is through node 2, where it is rejected
    toks, nodes = run(lg, tok, ptr, idx, q=[1, 1, 1, 1], u=[0, .6, .4, .5], us=.1)
    assert nodes == [0, 2]


def peaked(cfg, inp):
    """logits that put (numerically) all mass on the argmax of the generated logits"""
    am = oracle.argmax(inp["logits"])
    lg = np.full(inp["logits"].shape, -80.0, dtype=np.float32)
    np.put_along_axis(lg, am[..., None].astype(np.int64), 0.0, axis=-1)
    return lg


@pytest.mark.parametrize("name", ["tiny", "llama7b"])
def test_reduces_to_the_deterministic_rule_for_one_hot_targets(name):
    # with a one-hot target distribution, q = 1 and any u in (0, 1) the test "u < min(1, p/q)"
    # is "the token is the target's argmax", and the regenerated token is that argmax
    cfg = gi.CONFIGS[name]
    longest = 0
    for trial in range(4):
        inp = gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False)
        lg = peaked(cfg, inp)
        rng = np.random.default_rng(5 + trial)
        u = rng.uniform(0.01, 0.99, size=(cfg.B, cfg.N)).astype(np.float32)
        us = rng.uniform(0.01, 0.99, size=(cfg.B,)).astype(np.float32)
        q = np.ones((cfg.B, cfg.N), dtype=np.float32)
        t0, l0, n0, _ = oracle.accept(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
        t1, l1, n1 = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, u, us)
        assert (l0 == l1).all() and (t0 == t1).all() and (n0 == n1).all()
        longest = max(longest, int(l0.max()))
    assert longest > 1             # the generator plants agreement: some path is really accepted


def test_u_zero_accepts_every_step_with_mass_and_larger_u_never_helps():
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, attn=False)
    lg = inp["logits"]
    B, N = cfg.B, cfg.N
    q = np.full((B, N), 0.3, dtype=np.float32)
    us = np.full((B,), 0.5, dtype=np.float32)
    zero = np.zeros((B, N), dtype=np.float32)
    _, l_all, nodes_all = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q, zero, us)
    # every step accepted: the hypothesis is a longest root path of the graph = deepest level + 1
    for b in range(B):
        depth = max(inp["levels"][b])
        assert l_all[b] == depth + 1
    rng = np.random.default_rng(9)
    u = rng.uniform(0, 1, size=(B, N)).astype(np.float32)
    prev = l_all
    for scale in (0.25, 0.5, 1.0):
        _, l, _ = oracle.accept_sampled(lg, inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"], q,
                                        (u * scale).astype(np.float32), us)
        assert (l <= prev).all()
        prev = l


def test_acceptance_frequency_matches_min_one_p_over_q():
    # one step, many independent u: the fraction accepted is min(1, p/q) (Sec. 3)
    ptr, idx = chain(2)
    P = np.array([[.2, .8], [.5, .5]])
    n = 4000
    rng = np.random.default_rng(1)
    for q, want in ((.4, .5), (.1, 1.0), (.8, .25)):
        acc = 0
        for u in rng.uniform(0, 1, size=n):
            acc += len(run(LOG(P), [0, 0], ptr, idx, q=[1, q], u=[0, u], us=.3)[1]) == 2
        assert abs(acc / n - want) < 0.03


# ---- the regenerated token: residual of the sampling scheme that Sec. 3 cites ----

def run_res(logits, dlogits, tok, ptr, idx, q, u, us):
    t, l, nd = oracle.accept_sampled(np.asarray(logits, np.float32)[None], np.asarray(tok, np.int32)[None], ptr, idx,
                                     np.asarray(q, np.float32)[None], np.asarray(u, np.float32)[None],
                                     np.asarray([us], np.float32),
                                     draft_logits=None if dlogits is None else np.asarray(dlogits, np.float32)[None])
    n = int(l[0])
    return list(t[0, :n]), list(nd[0, :n])


def test_worked_residual():
    # root: P = [.4,.3,.2,.1], Q = [.1,.2,.3,.4]: max(0, P - Q) = [.3,.1,0,0], mass .4
    P = np.array([[.4, .3, .2, .1], [.25, .25, .25, .25]])
    Q = np.array([[.1, .2, .3, .4], [.25, .25, .25, .25]])
    ptr, idx = chain(2)
    # the child carries token 3 (p = .1, q = .4): u q = .9 * .4 = .36 is not below .1 -> rejected
    for us, want in ((.7, 0), (.74, 0), (.76, 1), (.99, 1), (0.0, 0)):
        toks, nodes = run_res(LOG(P), LOG(Q), [0, 3], ptr, idx, q=[1, .4], u=[0, .9], us=us)
        assert nodes == [0] and toks == [want], (us, toks)
    # without the draft distribution the token comes from P itself: cumulative .4, .7, .9, 1
    for us, want in ((.39, 0), (.41, 1), (.71, 2), (.95, 3)):
        assert run_res(LOG(P), None, [0, 3], ptr, idx, q=[1, .4], u=[0, .9], us=us)[0] == [want]
    # and the residual never yields a token to which the draft gives at least the target's mass
    for us in np.linspace(0, 0.999, 23):
        assert run_res(LOG(P), LOG(Q), [0, 3], ptr, idx, q=[1, .4], u=[0, .9], us=us)[0][0] in (0, 1)


def test_residual_is_formed_at_the_end_node():
    # chain 0 -> 1 -> 2: the first step is accepted, the second rejected; the residual is that of
    # node 1 (P1 - Q1 = [0, 0, .2, .2] -> tokens 2, 3), not of the root (tokens 0, 1)
    P = np.array([[.4, .3, .2, .1], [.1, .1, .4, .4], [.25] * 4])
    Q = np.array([[.1, .2, .3, .4], [.3, .3, .2, .2], [.25] * 4])
    ptr, idx = chain(3)
    for us, want in ((.3, 2), (.49, 2), (.51, 3), (.9, 3)):
        toks, nodes = run_res(LOG(P), LOG(Q), [0, 0, 1], ptr, idx, q=[1, .1, .3], u=[0, .5, .9], us=us)
        assert nodes == [0, 1] and toks == [0, want]


def test_no_rejection_at_the_end_node_draws_from_the_target():
    # the step 0 -> 1 is accepted and node 1 has no child: nothing was rejected there, so the
    # next token comes from P of node 1 whatever the draft distribution says
    P = np.array([[.4, .3, .2, .1], [.1, .2, .3, .4]])
    Q = np.array([[.1, .2, .3, .4], [.7, .1, .1, .1]])
    ptr, idx = chain(2)
    for us, want in ((.05, 0), (.2, 1), (.5, 2), (.7, 3)):
        toks, nodes = run_res(LOG(P), LOG(Q), [0, 0], ptr, idx, q=[1, .1], u=[0, .5], us=us)
        assert nodes == [0, 1] and toks == [0, want]


def test_residual_without_mass_falls_back_to_the_target():
    # draft distribution == target distribution: P - Q is zero everywhere; a rejection forced
    # through an inconsistent draft_q then regenerates from P
    P = np.array([[.5, .25, .125, .125], [.25, .25, .25, .25]])
    ptr, idx = chain(2)
    for us, want in ((.4, 0), (.6, 1), (.8, 2), (.9, 3)):
        toks, nodes = run_res(LOG(P), LOG(P), [0, 2], ptr, idx, q=[1, 1.0], u=[0, .5], us=us)
        assert nodes == [0] and toks == [want]


def test_rejected_siblings_share_one_residual():
    # the root has two children (tokens 2 and 3), both rejected; the residual is max(0, P - Q) of
    # the root, formed once: [.3, .1, 0, 0] / .4
    P = np.array([[.4, .3, .2, .1], [.25] * 4, [.25] * 4])
    Q = np.array([[.1, .2, .3, .4], [.25] * 4, [.25] * 4])
    ptr = np.array([[0, 0, 1, 2]], dtype=np.int32)
    idx = np.array([[0, 0]], dtype=np.int32)
    for us, want in ((.7, 0), (.8, 1)):
        toks, nodes = run_res(LOG(P), LOG(Q), [0, 2, 3], ptr, idx, q=[1, .3, .4], u=[0, .9, .9], us=us)
        assert nodes == [0] and toks == [want]
    # one of them accepted (u small): the hypothesis goes on and the leaf draws from its own P
    toks, nodes = run_res(LOG(P), LOG(Q), [0, 2, 3], ptr, idx, q=[1, .3, .4], u=[0, .9, .1], us=.6)
    assert nodes == [0, 2] and toks == [3, 2]


def chi_square(counts, probs):
    n = counts.sum()
    return float((((counts - n * probs) ** 2) / (n * probs)).sum())


def test_emitted_token_follows_the_target_distribution():
    # Sec. 3: the scheme "ensures that the tokens ultimately accepted are representative of the
    # output distribution of M_p".  One drafted token x ~ Q per sequence, seeded uniform numbers:
    # the first emitted token (x if accepted, else the regenerated one) must be distributed as P.
    # Bound: the 99.9 % point of chi-square with V - 1 = 5 degrees of freedom is 20.5.
    V, n = 6, 60000
    rng = np.random.default_rng(20240716)
    P = np.array([.30, .05, .25, .10, .02, .28])
    Q = np.array([.10, .25, .05, .30, .20, .10])
    x = rng.choice(V, size=n, p=Q)
    lg = np.empty((n, 2, V), dtype=np.float32)
    dl = np.empty((n, 2, V), dtype=np.float32)
    lg[:, 0] = LOG(P); lg[:, 1] = 0.0
    dl[:, 0] = LOG(Q); dl[:, 1] = 0.0
    tok = np.stack([np.zeros(n, np.int32), x.astype(np.int32)], axis=1)
    ptr = np.tile(np.array([0, 0, 1], dtype=np.int32), (n, 1))
    idx = np.zeros((n, 1), dtype=np.int32)
    q = np.stack([np.ones(n), Q[x]], axis=1).astype(np.float32)
    u = rng.uniform(0, 1, size=(n, 2)).astype(np.float32)
    us = rng.uniform(0, 1, size=n).astype(np.float32)
    t, l, _ = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us, draft_logits=dl)
    first = t[:, 0]
    counts = np.bincount(first, minlength=V).astype(np.float64)
    assert chi_square(counts, P) < 20.5
    # the accepted fraction is sum_x min(P, Q) and the rejected ones never emit a token with Q >= P
    assert abs((l == 2).mean() - np.minimum(P, Q).sum()) < 0.01
    assert set(np.unique(first[l == 1])) <= {0, 2, 5}
    # the same stream with the regenerated token drawn from P itself is visibly NOT distributed as P
    t2, _, _ = oracle.accept_sampled(lg, tok, ptr, idx, q, u, us)
    assert chi_square(np.bincount(t2[:, 0], minlength=V).astype(np.float64), P) > 1000
