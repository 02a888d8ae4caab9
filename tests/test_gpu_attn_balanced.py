"""gsd_verify_attn with the work shared out on the device from seq_lens (num_splits =
GSD_ATTN_SPLIT_BALANCED or GSD_ATTN_SPLIT_PER_SEQUENCE): same results as the
fp64 oracle, and a table that covers every key tile of every (sequence, kv head) pair exactly once."""
import numpy as np
import pytest
import torch

import gsd_inputs as gi
import oracle
from gpu_util import attn_tensors, out_to_f64
from plan_model import balanced_table, per_sequence_table

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3
BALANCED = -1
PER_SEQUENCE = -2
TCGEN05 = 2


def run(inp, **kw):
    import paper_2407_16207_b200 as gsd
    t = attn_tensors(inp)
    out = gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                              t["ancestor_mask"], t["seq_lens"], **kw)
    torch.cuda.synchronize()
    return out


def want_of(inp):
    return oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                       inp["ancestor_mask"], inp["seq_lens"])


def assert_close(got64, want):
    # (rows that see a handful of keys keep values of a few units, whose bf16 rounding step is
    # larger: the error is taken relative to max(1, |value|))
    assert np.isfinite(got64).all()
    err = np.abs(got64 - want) / np.maximum(1.0, np.abs(want))
    assert err.max() <= MAX_ABS, f"max-abs {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"mean-abs {err.mean():.3e}"


SHAPES = {
    # three row-tile items per (sequence, kv head), two draft tiles, lengths from nothing to 12 tiles
    "gqa_ragged": dict(B=5, Hq=8, Hkv=2, D=128, L=(0, 1500), N=130, depth=12, kmax=4, pmax=3),
    # three draft tiles, the last of them invisible to the first rows; no prefix at all
    "no_prefix": dict(B=3, Hq=4, Hkv=4, D=128, L=0, N=300, depth=14, kmax=4, pmax=3),
    # many more units per CTA than its look-up table holds
    "many_small_items": dict(B=300, Hq=8, Hkv=8, D=128, L=(0, 200), N=64, depth=8),
    # more sequences than the planning block has threads
    "many_sequences": dict(B=1100, Hq=1, Hkv=1, D=128, L=(0, 100), N=64, depth=8),
    # fewer tiles than the device has SMs
    "short_line": dict(B=2, Hq=1, Hkv=1, D=128, L=(5, 100), N=64, depth=6),
    # per-sequence plan: every sequence has 1.5 target lengths and is cut in two - 394 partial
    # results on a 148-SM device, two below what the workspace holds
    "near_the_slot_bound": dict(B=197, Hq=1, Hkv=1, D=128, L=1024, N=64, depth=6),
    # one long sequence among short ones: its items are cut into many pieces
    "one_long": dict(B=4, Hq=4, Hkv=1, D=128, L=(5000, 6000), N=128, depth=10),
}


def make(shape, seed=3):
    base = dict(name="t", config_id=7, kmax=3, pmax=2, V=8, vtok=8, p_agree=0.5)
    cfg = gi.VerifyConfig(**{**base, **SHAPES[shape]})
    inp = gi.make_inputs(cfg, seed, accept=False, pad_fill="nan")
    if shape == "one_long":
        # (only ever shortened: the rows behind a sequence's end hold NaN)
        inp["seq_lens"][:] = np.minimum(inp["seq_lens"], np.array([10, 1 << 20, 300, 77], dtype=np.int32))
    return cfg, inp


@pytest.mark.parametrize("mode", [BALANCED, PER_SEQUENCE])
@pytest.mark.parametrize("shape", sorted(SHAPES))
def test_balanced_against_the_oracle(shape, mode):
    cfg, inp = make(shape)
    got = run(inp, kernel=TCGEN05, num_splits=mode)
    assert_close(out_to_f64(got), want_of(inp))
    again = run(inp, kernel=TCGEN05, num_splits=mode)
    assert torch.equal(got, again)                            # bit-identical run to run
    # and within one bf16 step (2^-8 relative, values below 0.5 counted as 0.5) of the fixed plan's result
    fixed = run(inp, kernel=TCGEN05, num_splits=1).float()
    assert bool(((got.float() - fixed).abs() <= 2.0 ** -7 * fixed.abs().clamp(min=0.5)).all())


def test_balanced_is_chosen_on_request_only():
    import paper_2407_16207_b200 as gsd
    cfg = gi.CONFIGS["llama13b"]
    inp = gi.make_inputs(cfg, accept=False)
    dims = (cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, inp["Lmax"])
    assert gsd.gsd_verify_attn_num_splits(*dims) > 0
    assert gsd.gsd_verify_attn_num_splits(*dims, BALANCED) == BALANCED
    assert gsd.gsd_verify_attn_num_splits(*dims, PER_SEQUENCE) == PER_SEQUENCE
    assert gsd.gsd_verify_attn_num_splits(*dims, BALANCED, 1) >= 1          # the mma.sync kernel has no such plan
    assert gsd.gsd_verify_attn_num_splits(*dims, PER_SEQUENCE, 1) >= 1
    for mode in (BALANCED, PER_SEQUENCE):
        assert_close(out_to_f64(run(inp, num_splits=mode)), want_of(inp))
        assert_close(out_to_f64(run(inp, num_splits=mode, kernel=1)), want_of(inp))


def table_of(ws, ctas, items, B):
    """The planning kernel's table behind the partial results (layout of the tcgen05 back end:
    2 * ctas slots of 256 rows; then header, per-group runs, merge list, units, line offsets)."""
    def up(x):
        return (x + 255) // 256 * 256
    at = up(2 * ctas * 256 * 128 * 4) + up(2 * ctas * 256 * 2 * 4)
    raw = ws.cpu().numpy()
    def take(nbytes):
        nonlocal at
        a = raw[at:at + nbytes].view(np.int32)
        at += up(nbytes)
        return a
    hdr = take(256)
    cta = take(ctas * 8).reshape(ctas, 2)
    merge = take(ctas * 16).reshape(ctas, 4)
    units = take((items + ctas) * 16).reshape(items + ctas, 4)
    off = take((B + 1) * 4)
    return hdr, cta, merge, units, off


@pytest.mark.parametrize("shape", ["gqa_ragged", "one_long", "many_small_items", "short_line"])
def test_the_table_covers_every_tile_once(shape):
    import paper_2407_16207_b200 as gsd
    cfg, inp = make(shape, seed=11)
    t = attn_tensors(inp)
    Lmax = inp["Lmax"]
    need = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax, BALANCED, TCGEN05)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], t["ancestor_mask"],
                        t["seq_lens"], kernel=TCGEN05, num_splits=BALANCED, workspace=ws)
    torch.cuda.synchronize()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    G = cfg.Hq // cfg.Hkv
    tpu = (cfg.N * G + 255) // 256            # row-tile items of a (sequence, kv head) pair: CTAs of a group
    per_seq = cfg.Hkv
    pairs = cfg.B * per_seq
    nd = (cfg.N + 127) // 128
    line_max = pairs * ((Lmax + 127) // 128 + nd)
    groups = min(sms // tpu, line_max)
    hdr, cta, merge, units, off = table_of(ws, groups * tpu, pairs * tpu, cfg.B)
    T = [(int(min(max(L, 0), Lmax)) + 127) // 128 + nd for L in inp["seq_lens"]]
    total = per_seq * sum(T)
    assert hdr[1] == total and off[cfg.B] == total
    share = int(hdr[2])
    assert share == max(1, -(-total // groups))
    covered = {}
    slots_of = {}
    n_units = 0
    for k in range(groups):
        first, n = int(cta[k, 0]), int(cta[k, 1])
        assert first == n_units
        n_units += n
        tiles = 0
        for pair, t0, t1, slot in units[first:first + n]:
            Ti = T[pair // per_seq]
            assert 0 <= t0 < t1 <= Ti
            tiles += t1 - t0
            for tt in range(t0, t1):
                assert (pair, tt) not in covered
                covered[(pair, tt)] = k
            whole = t0 == 0 and t1 == Ti
            assert (slot == -1) == whole
            if not whole:
                slots_of.setdefault(int(pair), []).append(int(slot))
        assert tiles <= share
    assert len(covered) == total
    # entry by entry what the plain-Python model of the plan says
    model = balanced_table(inp["seq_lens"], Lmax, per_seq, nd, groups)
    assert (int(hdr[1]), share) == (model["total"], model["share"])
    assert [tuple(int(x) for x in r) for r in cta[:groups]] == model["runs"]
    assert [tuple(int(x) for x in u) for u in units[:n_units]] == model["units"]
    assert [tuple(int(x) for x in r[:3]) for r in merge[:hdr[0]]] == model["merge"]
    # the cut pairs, each with a run of consecutive slots in tile order
    assert hdr[0] == len(slots_of)
    listed = {int(r[0]): (int(r[1]), int(r[2])) for r in merge[:hdr[0]]}
    assert set(listed) == set(slots_of)
    all_slots = []
    for pair, sl in slots_of.items():
        assert len(sl) >= 2
        assert sl == list(range(sl[0], sl[0] + len(sl)))
        assert listed[pair] == (sl[0], len(sl))
        all_slots += sl
    assert len(set(all_slots)) == len(all_slots) and (not all_slots or max(all_slots) < 2 * groups)


@pytest.mark.parametrize("shape", ["gqa_ragged", "one_long", "many_sequences", "no_prefix", "near_the_slot_bound"])
def test_the_split_counts_follow_the_lengths(shape):
    """Per-sequence plan: the table behind the partial results holds, per sequence, a split
    count = its tile count over the common target (rounded, 1..32), and running unit and slot
    offsets that match those counts."""
    import paper_2407_16207_b200 as gsd
    cfg, inp = make(shape, seed=13)
    t = attn_tensors(inp)
    Lmax = max(inp["Lmax"], 1)          # (the cache tensor has at least one row)
    need = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax, PER_SEQUENCE, TCGEN05)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"], t["ancestor_mask"],
                        t["seq_lens"], kernel=TCGEN05, num_splits=PER_SEQUENCE, workspace=ws)
    torch.cuda.synchronize()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    G = cfg.Hq // cfg.Hkv
    tpu = (cfg.N * G + 255) // 256
    per_seq = cfg.Hkv * tpu
    items = cfg.B * per_seq
    nd = (cfg.N + 127) // 128
    slots = min((4 * 2 * sms + 2) // 3 + 1, items * 32)          # the host's bound on the partial results

    def up(x):
        return (x + 255) // 256 * 256
    at = up(slots * 256 * 128 * 4) + up(slots * 256 * 2 * 4)
    raw = ws.cpu().numpy()
    row = up((cfg.B + 1) * 4)
    hdr = raw[at:at + 12].view(np.int32)
    nsplit = raw[at + 256:at + 256 + cfg.B * 4].view(np.int32)
    unit_off = raw[at + 256 + row:at + 256 + row + (cfg.B + 1) * 4].view(np.int32)
    slot_off = raw[at + 256 + 2 * row:at + 256 + 2 * row + (cfg.B + 1) * 4].view(np.int32)
    model = per_sequence_table(inp["seq_lens"], Lmax, per_seq, nd, 2 * sms)
    assert (int(hdr[1]), int(hdr[2])) == (model["total"], model["target"])
    assert nsplit.tolist() == model["nsplit"]
    assert unit_off.tolist() == model["unit_off"]
    assert slot_off.tolist() == model["slot_off"]
    assert hdr[0] == unit_off[-1] and slot_off[-1] <= slots

