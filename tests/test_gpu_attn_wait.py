"""The bounded waits of the tcgen05 attention kernel: a wait that runs out must end the launch
cleanly with GSD_DEV_WAIT_EXPIRED, and the next call must work as if nothing had happened.

The wait is made to run out through the library's test hook: with a limit of a few milliseconds
every CTA announces the copy of its first key tile but never issues it (nothing is broken on
purpose beyond that: every other copy is issued, every wait keeps its limit, nothing traps)."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import attn_tensors, out_to_f64

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_next_call_is_clean():
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["llama7b"]
    inp = gi.make_inputs(cfg, accept=False)
    t = attn_tensors(inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def call():
        out = gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                                  t["ancestor_mask"], t["seq_lens"], kernel=gsd.GSD_ATTN_TCGEN05, status=status)
        torch.cuda.synchronize()
        return out

    gsd.gsd_debug_attn_wait(3_000_000, True)          # 3 ms instead of 2 s; first K tile withheld
    try:
        call()
        assert int(status.item()) & 0x8               # GSD_DEV_WAIT_EXPIRED
    finally:
        gsd.gsd_debug_attn_wait(0, False)
    # the context is intact and the kernel's resources were given back: an ordinary call is right
    status.zero_()
    out = call()
    assert int(status.item()) == 0
    want = oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                       inp["ancestor_mask"], inp["seq_lens"])
    err = np.abs(out_to_f64(out) - want)
    assert err.max() <= 1e-2 and err.mean() <= 1e-3
    # and once more on the configuration with two row tiles per unit and several units per CTA
    cfg = gi.sweep_config(1, 512, 512)
    inp = gi.make_inputs(cfg, accept=False)
    t2 = attn_tensors(inp)
    gsd.gsd_debug_attn_wait(3_000_000, True)
    try:
        gsd.gsd_verify_attn(t2["q"], t2["k_cache"], t2["v_cache"], t2["draft_k"], t2["draft_v"],
                            t2["ancestor_mask"], t2["seq_lens"], status=status)
        torch.cuda.synchronize()
        assert int(status.item()) & 0x8
    finally:
        gsd.gsd_debug_attn_wait(0, False)
    status.zero_()
    out = gsd.gsd_verify_attn(t2["q"], t2["k_cache"], t2["v_cache"], t2["draft_k"], t2["draft_v"],
                              t2["ancestor_mask"], t2["seq_lens"], status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = [(0, n, h) for n in range(0, cfg.N, 37) for h in range(0, cfg.Hq, 5)]
    want = oracle.attn_rows(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                            inp["ancestor_mask"], inp["seq_lens"], rows)
    got = np.stack([out_to_f64(out[b, n, h]) for b, n, h in rows])
    assert np.abs(got - want).max() <= 1e-2
