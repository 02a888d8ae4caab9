"""gsd_commit_kv on the GPU against the oracle: a copy of whole rows, compared bit for bit."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import accept_tensors, bf16_bits, bf16_tensor, i32_tensor

pytestmark = pytest.mark.gpu


def run_both(inp, kc, vc, sl, nodes, lens, status=None):
    import paper_2407_16207_b200 as gsd
    dk, dv = inp["draft_k"], inp["draft_v"]
    want = oracle.commit_kv(kc, vc, dk, dv, nodes, lens, sl)
    k = bf16_tensor(kc, "cuda"); v = bf16_tensor(vc, "cuda")
    s = i32_tensor(sl, "cuda").clone()
    gsd.gsd_commit_kv(k, v, bf16_tensor(dk, "cuda"), bf16_tensor(dv, "cuda"), i32_tensor(nodes, "cuda"),
                      i32_tensor(lens, "cuda"), s, status=status)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(k), want[0])
    assert np.array_equal(bf16_bits(v), want[1])
    assert np.array_equal(s.cpu().numpy(), want[2])
    return want


@pytest.mark.parametrize("name", ["tiny", "llama7b", "llama13b", "llama70b"])
def test_commit_after_accept_bit_exact(name):
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS[name]
    inp = gi.make_inputs(cfg)
    grow = cfg.depth + 1
    pad = np.full((cfg.B, grow, cfg.Hkv, cfg.D), 0x7FC0, dtype=np.uint16)
    kc = np.concatenate([inp["k_cache"], pad], axis=1)
    vc = np.concatenate([inp["v_cache"], pad], axis=1)
    t = accept_tensors(inp)
    toks, lens, nodes = gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"])
    want = run_both(inp, kc, vc, inp["seq_lens"], nodes.cpu().numpy(), lens.cpu().numpy())
    assert want[3] == 0 and np.array_equal(want[2], inp["seq_lens"] + lens.cpu().numpy())


def test_overflow_bad_nodes_and_flags():
    cfg = gi.VerifyConfig("t", 9, 3, 4, 2, 64, 20, 9, 3, 3, 2, 16, 16, 0.5)
    inp = gi.make_inputs(cfg, accept=False)
    kc, vc = inp["k_cache"].copy(), inp["v_cache"].copy()
    nodes = np.array([[0, 1, 2, 3, -1, -1], [0, 99, 4, -1, -1, -1], [0, 5, -1, -1, -1, -1]], dtype=np.int32)
    lens = np.array([4, 3, 2], dtype=np.int32)
    sl = np.array([18, 5, 20], dtype=np.int32)                    # room for 2, plenty, none
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want = run_both(inp, kc, vc, sl, nodes, lens, status=status)
    assert list(want[2]) == [20, 7, 20]
    assert int(status.item()) == (0x20 | 0x1)
