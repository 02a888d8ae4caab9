"""The two work plans that gsd_verify_attn makes on the device from seq_lens, written out in plain
Python from their definition (a model for the tests; the library does not use it).

Balanced plan: the key tiles of all (sequence, kv head) pairs lie end to end on a line - pair after
pair, ceil(len / 128) prefix tiles plus `nd` draft tiles each - and group g of `groups` takes the
g-th share of ceil(total / groups) tiles.  A unit is the piece of one pair inside one share; pieces
that are not a whole pair get consecutive partial-result slots along the line.

Per-sequence plan: every pair of sequence b is cut into n_b = round(T_b / target) ranges (1..32),
target = max(4, ceil(total item tiles / units_wanted)); units and slots are numbered sequence by
sequence."""
from typing import Dict, List, Tuple


def tiles_of(seq_lens, Lmax: int, nd: int) -> List[int]:
    return [(min(max(int(L), 0), Lmax) + 127) // 128 + nd for L in seq_lens]


def balanced_table(seq_lens, Lmax: int, per_seq: int, nd: int, groups: int) -> Dict[str, object]:
    T = tiles_of(seq_lens, Lmax, nd)
    line: List[Tuple[int, int]] = []          # (pair, tile) in line order
    for b, t in enumerate(T):
        for c in range(per_seq):
            line += [(b * per_seq + c, k) for k in range(t)]
    total = len(line)
    share = max(1, -(-total // groups))
    units: List[Tuple[int, int, int, int]] = []   # (pair, first tile, end tile, slot or -1)
    runs: List[Tuple[int, int]] = []              # per group: (first unit, units)
    slot = 0
    for g in range(groups):
        piece = line[min(g * share, total):min((g + 1) * share, total)]
        first = len(units)
        i = 0
        while i < len(piece):
            pair, t0 = piece[i]
            j = i
            while j < len(piece) and piece[j][0] == pair:
                j += 1
            t1 = piece[j - 1][1] + 1
            whole = t0 == 0 and t1 == T[pair // per_seq]
            units.append((pair, t0, t1, -1 if whole else slot))
            slot += 0 if whole else 1
            i = j
        runs.append((first, len(units) - first))
    merge: List[Tuple[int, int, int]] = []        # (pair, first slot, slots) of every cut pair, in line order
    seen: Dict[int, List[int]] = {}
    for pair, _, _, s in units:
        if s >= 0:
            seen.setdefault(pair, []).append(s)
    for pair in sorted(seen):
        merge.append((pair, seen[pair][0], len(seen[pair])))
    return {"total": total, "share": share, "units": units, "runs": runs, "merge": merge, "slots": slot}


def per_sequence_table(seq_lens, Lmax: int, per_seq: int, nd: int, units_wanted: int) -> Dict[str, object]:
    T = tiles_of(seq_lens, Lmax, nd)
    total = per_seq * sum(T)
    target = max(4, -(-total // units_wanted))
    nsplit = [min(32, max(1, (2 * t + target) // (2 * target))) for t in T]
    unit_off, slot_off = [0], [0]
    for n in nsplit:
        unit_off.append(unit_off[-1] + n * per_seq)
        slot_off.append(slot_off[-1] + (n * per_seq if n > 1 else 0))
    return {"total": total, "target": target, "nsplit": nsplit, "unit_off": unit_off, "slot_off": slot_off}
