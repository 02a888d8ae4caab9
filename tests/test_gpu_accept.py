"""gsd_accept on the GPU against the CPU oracle: bit-exact tokens, lengths and node paths."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, i32_tensor
from helpers import load_accept_cases, logits_with_argmax

pytestmark = pytest.mark.gpu


def run_gpu(inp_np, Tcap=0, status=None):
    import paper_2407_16207_b200 as gsd
    t = accept_tensors(inp_np)
    toks, lens, nodes = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"],
                                       t["parent_idx"], Tcap=Tcap, status=status)
    torch.cuda.synchronize()
    return toks.cpu().numpy(), lens.cpu().numpy(), nodes.cpu().numpy()


def check_against_oracle(inp, Tcap=0):
    want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"],
                         Tcap=Tcap)
    got = run_gpu(inp, Tcap=Tcap)
    assert np.array_equal(got[1], want[1])
    assert np.array_equal(got[0], want[0])
    assert np.array_equal(got[2], want[2])


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
@pytest.mark.parametrize("trial", [0, 1, 2])
def test_configs_bit_exact(name, trial):
    cfg = gi.CONFIGS[name]
    check_against_oracle(gi.make_inputs(cfg, gi.seed_for(cfg, trial), attn=False))


def test_sweep_point_512_nodes():
    cfg = gi.sweep_config(2, 512, 512)
    inp = gi.make_inputs(cfg, attn=False)
    want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"],
                         visit_cap=5_000_000)
    got = run_gpu(inp)
    for g, w in zip(got, want[:3]):
        assert np.array_equal(g, w)


def test_hand_built_dags():
    for case in load_accept_cases():
        ptr, idx = gi.parents_to_csr([case["parents"]])
        inp = dict(logits=logits_with_argmax(case["argmax"], 128)[None],
                   draft_tokens=np.array([case["tokens"]], dtype=np.int32),
                   parent_ptr=ptr, parent_idx=idx)
        toks, lens, nodes = run_gpu(inp)
        m = int(lens[0])
        assert list(toks[0, :m]) == case["expect_tokens"], case["name"]
        assert list(nodes[0, :m]) == case["expect_nodes"], case["name"]
        assert (toks[0, m:] == -1).all() and (nodes[0, m:] == -1).all()


@pytest.mark.parametrize("V", [1, 3, 4, 1000, 4099, 32000, 65536 + 4])
def test_argmax_ties_nan_inf_and_odd_vocab(V):
    # single-node sequences: accepted_tokens[b, 0] is the argmax of row b
    rng = np.random.default_rng(V)
    B = 24
    x = rng.standard_normal((B, 1, V)).astype(np.float32)
    if V >= 4:
        x[0, 0, [0, V // 2, V - 1]] = 9.0                       # ties across slices / lanes
        x[1, 0, :] = 1.25
        x[2, 0, V - 1] = 30.0
        x[3, 0, :] = -np.inf
        x[4, 0, :] = np.nan
        x[5, 0, :] = np.nan; x[5, 0, V - 2] = -np.inf
        x[6, 0, :] = -0.0; x[6, 0, V - 1] = 0.0
        x[7, 0, 1] = np.inf; x[7, 0, 3] = np.inf
        x[8, 0, 0] = np.nan; x[8, 0, 1:] = -3.0
        for b in range(9, 16):                                    # equal maxima 1 apart, all offsets
            x[b, 0, (b * 37) % V] = 11.0
            x[b, 0, ((b * 37) % V + 1) % V] = 11.0
    inp = dict(logits=x, draft_tokens=np.zeros((B, 1), dtype=np.int32),
               parent_ptr=np.zeros((B, 2), dtype=np.int32),
               parent_idx=np.full((B, 1), -1, dtype=np.int32))
    toks, lens, _ = run_gpu(inp)
    assert (lens == 1).all()
    assert np.array_equal(toks[:, 0], oracle.argmax(x)[:, 0])


def test_unaligned_logits_take_the_scalar_path():
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["tiny"]
    inp = gi.make_inputs(cfg, attn=False)
    t = accept_tensors(inp)
    flat = torch.empty(t["logits"].numel() + 1, dtype=torch.float32, device="cuda")
    shifted = flat[1:].view_as(t["logits"])
    shifted.copy_(t["logits"])
    assert shifted.data_ptr() % 16 != 0
    toks, lens, nodes = gsd.gsd_accept(shifted, t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
    want = oracle.accept(inp["logits"], inp["draft_tokens"], inp["parent_ptr"], inp["parent_idx"])
    assert np.array_equal(toks.cpu().numpy(), want[0])
    assert np.array_equal(lens.cpu().numpy(), want[1])


def test_device_status_flags_and_clean_finish():
    # a parent index that is not below its child is ignored and flagged; no trap
    tok = np.array([[0, 5, 6]], dtype=np.int32)
    ptr = np.array([[0, 0, 1, 2]], dtype=np.int32)
    idx = np.array([[0, 2]], dtype=np.int32)          # node 2 names itself as parent
    inp = dict(logits=logits_with_argmax([5, 6, 7], 16)[None], draft_tokens=tok,
               parent_ptr=ptr, parent_idx=idx)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    toks, lens, nodes = run_gpu(inp, status=status)
    assert int(status.item()) & 0x1
    assert lens[0] == 2 and list(toks[0, :2]) == [5, 6] and list(nodes[0, :2]) == [0, 1]
    # token outside the vocabulary: flagged, still compared as is
    inp["parent_idx"] = np.array([[0, 1]], dtype=np.int32)
    inp["draft_tokens"] = np.array([[0, 5, 99]], dtype=np.int32)
    status.zero_()
    toks, lens, _ = run_gpu(inp, status=status)
    assert int(status.item()) == 0x2 and lens[0] == 2
    # capacity: Tcap 2 cannot hold 3 tokens -> truncated and flagged, length still reported
    inp["draft_tokens"] = tok
    status.zero_()
    toks, lens, _ = run_gpu(inp, Tcap=2, status=status)
    assert int(status.item()) == 0x4 and lens[0] == 3 and list(toks[0]) == [5, 6]


def test_repeated_calls_are_identical():
    cfg = gi.CONFIGS["llama13b"]
    inp = gi.make_inputs(cfg, attn=False)
    a = run_gpu(inp)
    b = run_gpu(inp)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_more_rows_than_one_launch_holds():
    # B * N = 70400 rows: the library sends them out as two launches of whole sequences (a grid
    # dimension holds 65535 rows); results and the per-sequence completion counters must not care
    cfg = gi.VerifyConfig("many", 6, 1100, 1, 1, 64, 8, 64, 8, 3, 2, 128, 128, 0.7)
    inp = gi.make_inputs(cfg, attn=False)
    assert cfg.B * cfg.N > 65535
    check_against_oracle(inp)


def sanitised_parents(ptr, idx, N):
    """What the library documents for row pointers that do not start at zero or go backwards:
    they are replaced by their running maximum (from zero), and parent indices outside [0, v)
    are ignored.  Written out here in plain Python."""
    run, sp = 0, [0]
    for v in range(1, N + 1):
        run = max(run, min(max(int(ptr[v]), 0), len(idx)))
        sp.append(run)
    return [[int(p) for p in idx[sp[v]:sp[v + 1]] if 0 <= p < v] for v in range(N)]


@pytest.mark.parametrize("ptr", [
    [0, 0, 1, 5, 3, 4, 6],        # an interior pointer above the last one, then going backwards
    [2, 2, 3, 4, 5, 6, 6],        # does not start at zero: edges 0, 1 belong to the root's row and are ignored
    [0, 0, 4, 2, 3, 9, 5],        # a pointer past the capacity (clamped) and non-monotone ones
])
def test_row_pointers_that_go_backwards_are_flagged_and_made_safe(ptr):
    N, Ecap = 6, 8
    idx = np.array([[0, 0, 1, 1, 2, 3, 4, 2]], dtype=np.int32)
    tok = np.array([[0, 5, 6, 7, 8, 9]], dtype=np.int32)
    logits = logits_with_argmax([5, 6, 7, 8, 9, 3], 16)[None]          # node v's argmax is the token of node v+1
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    inp = dict(logits=logits, draft_tokens=tok, parent_ptr=np.array([ptr], dtype=np.int32), parent_idx=idx)
    got = run_gpu(inp, status=status)
    assert int(status.item()) & 0x1
    parents = sanitised_parents(ptr, idx[0], N)
    cptr, cidx = gi.parents_to_csr([parents], Ecap)
    want = oracle.accept(logits, tok, cptr, cidx)
    for g, w in zip(got, want[:3]):
        assert np.array_equal(g, w)
