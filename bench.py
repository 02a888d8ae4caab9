#!/usr/bin/env python
"""Benchmark of the GSD verification step (gsd_verify_attn + gsd_accept) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
  python bench.py --sweep [--points B1_L512_N32,...]      one JSON line per point of the 70B-shaped sweep
  python bench.py --ab-unmerge                             graph-direct vs unmerged-tree verification

A step is one pass of the whole hot path over one batch of synthetic LLaMA-2-shaped input:
DAG-masked attention of all draft nodes, then vocabulary argmax and longest accepted path.
NAME is tiny, llama7b, llama13b, llama70b (default) or a sweep point sweep_B{b}_L{l}_N{n}.
Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent replica of the
workload (the path has no cross-GPU exchange), timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import gsd_inputs as gi  # noqa: E402

METRIC = "draft_tokens_verified_per_s_per_attn_layer"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
L2_BYTES = 126 << 20
SWEEP_B, SWEEP_L, SWEEP_N = (1, 8, 32), (512, 2048, 8192, 32768), (32, 128, 512)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def config_by_name(name: str) -> gi.VerifyConfig:
    if name in gi.CONFIGS:
        return gi.CONFIGS[name]
    m = re.fullmatch(r"(?:sweep_)?B(\d+)_L(\d+)_N(\d+)", name)
    if not m:
        raise SystemExit(f"unknown workload {name!r}: one of {sorted(gi.CONFIGS)} or sweep_B<b>_L<l>_N<n>")
    return gi.sweep_config(int(m.group(1)), int(m.group(2)), int(m.group(3)))


def algorithmic_work(cfg, inp):
    """Algorithmic flops and bytes of one gsd_verify_attn call and bytes of one gsd_accept call.

    flops: 4 * Hq * D per (node, visible key): prefix keys seq_lens[b] plus the set mask bits.
    bytes: K and V of the visible prefix and of the draft block once per kv head, Q in and
    out once, the mask once; accept reads the logits once."""
    B, N, Hq, Hkv, D = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D
    L = inp["seq_lens"].astype(np.int64)
    bits = np.unpackbits(inp["ancestor_mask"].view(np.uint8), axis=-1).reshape(B, N, -1).sum(-1)
    visible = (L[:, None] + bits).sum()
    flops = 4.0 * Hq * D * float(visible)
    kv_bytes = 2 * 2 * D * Hkv * float((L + N).sum())
    qo_bytes = 2 * 2 * D * Hq * B * N
    mask_bytes = inp["ancestor_mask"].nbytes
    accept_bytes = 4.0 * B * N * cfg.V
    return flops, kv_bytes + qo_bytes + mask_bytes, accept_bytes


def roofline_of(flops, attn_bytes, seconds, peaks, peak_src):
    """The roofline object of one gsd_verify_attn call that took `seconds`.  One fixed pair of
    denominators: the measured burst bf16 throughput and the measured copy bandwidth."""
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = attn_bytes / (peaks["hbm_gbs"] * 1e9)
    if t_tc >= t_hbm:
        achieved = flops / seconds / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "traffic": None,
                "peak_kind": f"burst bf16, of {peak_src}",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_nominal": achieved / NOMINAL["bf16_tflops"]}
    else:
        achieved = attn_bytes / seconds / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                "peak_kind": f"copy bandwidth, of {peak_src}",
                "frac_of_nominal": achieved / NOMINAL["hbm_gbs"]}
    roof["roofline_us"] = max(t_tc, t_hbm) * 1e6
    roof["algorithmic_flops"] = flops
    roof["algorithmic_bytes"] = attn_bytes
    return roof


def recorded_traffic(kernel_name: str, workload: str):
    """DRAM bytes per launch of `kernel_name` on `workload` as recorded beside the ncu summaries
    (kernel, workload, bytes, and the SHA-256 of the kernel's source at capture time).  None when
    there is no record or the source has changed since: the counters then describe other code."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        lines = open(path).read().splitlines()
    except OSError:
        return None
    for line in lines:
        f = line.split()
        if len(f) == 5 and not line.startswith("#") and f[0] == kernel_name and f[1] == workload:
            src = os.path.join(ROOT, "paper_2407_16207_b200", "csrc", f[3])
            try:
                digest = hashlib.sha256(open(src, "rb").read()).hexdigest()
            except OSError:
                return None
            return float(f[2]) if digest == f[4] else None
    return None


class ClockSampler:
    """Samples the SM clock and the throttle reasons (read-only NVML queries) from a thread
    while the timed region runs."""
    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
               "sw_power_cap": 0x4}

    def __init__(self, index: int):
        import threading
        self.sm, self.reasons, self.max_mhz, self.err = [], set(), None, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
        except Exception as e:  # pragma: no cover
            self.err = f"NVML unavailable: {e}"

    def start(self):
        if self._thread:
            self._thread.start()

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for name, bit in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception as e:  # pragma: no cover
                self.err = str(e)
                return
            self._stop.wait(0.002)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        out = {"sm_mhz": statistics.median(self.sm) if self.sm else None,
               "sm_max_mhz": self.max_mhz, "samples": len(self.sm), "reasons": sorted(self.reasons)}
        if self.err:
            out["note"] = self.err
        return out


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return rank, world, local, dist
    torch.cuda.set_device(local)
    return rank, world, local, None


def aggregate_over_ranks(ms_per_step, tokens_per_step, world, dist, device):
    """Step time = the maximum over ranks; value = the tokens of all replicas over that time."""
    if dist is not None and world > 1:
        tt = torch.tensor([ms_per_step], dtype=torch.float64, device=device)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_per_step = float(tt.item())
    return {"ms_per_step": ms_per_step, "value": world * tokens_per_step / (ms_per_step * 1e-3)}


# ------------------------------------------------------------------------------ CPU oracle legs
def cpu_oracle_time(cfg, inp, rows: int, accept_seqs: int = 0):
    """Times the CPU oracle (as it stands) on the workload: `rows` consecutive attention rows
    (all of them when rows >= B*N*Hq; otherwise a block starting at a seeded offset, the same
    access pattern as the full run) plus the acceptance of `accept_seqs` sequences (0 = all).
    Returns a cpu_baseline object; anything not run in full is scaled up and says so."""
    import oracle
    total_rows = cfg.B * cfg.N * cfg.Hq
    n = int(min(max(rows, 1), total_rows))
    t0 = time.perf_counter()
    if n == total_rows:
        oracle.attn(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                    inp["ancestor_mask"], inp["seq_lens"])
    else:
        r0 = int(np.random.default_rng(0).integers(0, total_rows - n + 1))
        r = np.arange(r0, r0 + n)
        rows_bnh = np.stack([r // (cfg.N * cfg.Hq), (r // cfg.Hq) % cfg.N, r % cfg.Hq], axis=1).astype(np.int32)
        oracle.attn_rows(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                         inp["ancestor_mask"], inp["seq_lens"], rows_bnh)
    t_attn = time.perf_counter() - t0
    nb = cfg.B if accept_seqs <= 0 else min(accept_seqs, cfg.B)
    t0 = time.perf_counter()
    oracle.accept(inp["logits"][:nb], inp["draft_tokens"][:nb], inp["parent_ptr"][:nb], inp["parent_idx"][:nb],
                  visit_cap=5_000_000)
    t_acc = time.perf_counter() - t0
    t_step = t_attn * (total_rows / n) + t_acc * (cfg.B / nb)
    full = n == total_rows and nb == cfg.B
    desc = (f"{'all' if n == total_rows else n} of {total_rows} attention rows ({t_attn:.3f} s) + acceptance of "
            f"{nb} of {cfg.B} sequences ({t_acc:.3f} s)" + ("" if full else "; scaled to the whole step"))
    return {"value": cfg.B * cfg.N / t_step, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": desc, "extrapolated": not full, "sampled_fraction": n / total_rows,
            "seconds_per_step": t_step}


def run_reference(args, cfg):
    """The reference arm: the CPU oracle, timed on the host cores.  A step is the whole workload
    when K + W such steps fit in about two minutes; otherwise each step is a block of rows sized
    for that budget and the line says that its value is extrapolated."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = gi.make_inputs(cfg)
    total_rows = cfg.B * cfg.N * cfg.Hq
    n_steps = args.warmup + args.steps
    probe = cpu_oracle_time(cfg, inp, min(total_rows, 8192), 1)          # calibration, not reported
    budget_s = 120.0
    rows_per_step = int(min(total_rows, max(64, total_rows * budget_s / (n_steps * probe["seconds_per_step"]))))
    if rows_per_step > 0.9 * total_rows:
        rows_per_step = total_rows
    accept_seqs = 0 if rows_per_step == total_rows else 1
    runs = []
    for i in range(n_steps):
        r = cpu_oracle_time(cfg, inp, rows_per_step, accept_seqs)
        if i >= args.warmup:
            runs.append(r)
    sec = sum(r["seconds_per_step"] for r in runs) / len(runs)
    value = cfg.B * cfg.N / sec
    last = runs[-1]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "extrapolated": last["extrapolated"],
            "sampled_fraction": last["sampled_fraction"],
            "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv,
                       "D": cfg.D, "L": cfg.L, "V": cfg.V},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                             "sample": "per step: " + last["sample"], "extrapolated": last["extrapolated"],
                             "sampled_fraction": last["sampled_fraction"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ the 70B-shaped sweep
def run_sweep(args):
    """One JSON line per point: gsd_verify_attn (automatic kernel choice) and gsd_accept on the
    seeded inputs of that point, timed cold (a buffer larger than L2 is written between calls)
    and warm (the same resident set called back to back), each against the roofline."""
    import paper_2407_16207_b200 as gsd
    from gsd_inputs.torch_io import accept_tensors, attn_tensors
    gsd.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks, peak_src = load_peaks()
    if args.points:
        names = args.points.split(",")
    else:
        names = ["llama7b", "llama13b", "llama70b"] + [f"sweep_B{b}_L{l}_N{n}" for b in SWEEP_B for l in SWEEP_L
                                                       for n in SWEEP_N]
    flush = torch.empty(4 * L2_BYTES, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    reps = max(args.steps if args.steps_given else 20, 3)
    prev = None
    for name in names:
        cfg = config_by_name(name)
        reuse = prev if (prev is not None and prev["cfg"].name.startswith("sweep") and name.startswith("sweep")
                         and (prev["cfg"].B, prev["cfg"].L) == (cfg.B, cfg.L)) else None
        inp = gi.make_inputs(cfg, kv_from=reuse)
        prev = inp
        t = {**attn_tensors(inp, dev), **accept_tensors(inp, dev)}
        out = torch.empty_like(t["q"])
        Lmax = inp["Lmax"]
        ws = torch.empty(max(gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax), 256),
                         dtype=torch.uint8, device=dev)
        ws_acc = torch.empty(gsd.gsd_accept_workspace_bytes(cfg.B, cfg.N), dtype=torch.uint8, device=dev)
        acc_out = (torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=dev),
                   torch.empty((cfg.B,), dtype=torch.int32, device=dev),
                   torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=dev))

        def attn():
            gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                                t["ancestor_mask"], t["seq_lens"], out=out, workspace=ws, status=status)

        def accept():
            gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"],
                           workspace=ws_acc, status=status, out=acc_out)

        for _ in range(3):
            attn(); accept()
        torch.cuda.synchronize()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(reps)]
        for i in range(reps):                       # cold: L2 holds the flush buffer's lines
            flush.fill_(i & 0xFF)
            ev[i][0].record(); attn(); ev[i][1].record(); accept(); ev[i][2].record()
        torch.cuda.synchronize()
        attn_cold = statistics.median(e[0].elapsed_time(e[1]) for e in ev) * 1e-3
        acc_cold = statistics.median(e[1].elapsed_time(e[2]) for e in ev) * 1e-3
        # warm: the calls are captured in CUDA graphs and replayed, so that the host's launch work
        # (which would bound calls of a few microseconds) is not in the numbers
        def graph_time(fn):
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for _ in range(reps):
                        fn()
            torch.cuda.current_stream().wait_stream(side)
            g.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); g.replay(); b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) * 1e-3 / reps
        attn_warm = graph_time(attn)
        acc_warm = graph_time(accept)
        if int(status.item()) != 0:
            raise RuntimeError(f"device status {int(status.item()):#x} on {name}")
        flops, attn_bytes, accept_bytes = algorithmic_work(cfg, inp)
        roof = roofline_of(flops, attn_bytes, attn_cold, peaks, peak_src)
        roof["kernel"] = "gsd_verify_attn"
        roof["frac_warm"] = roofline_of(flops, attn_bytes, attn_warm, peaks, peak_src)["frac"]
        tokens = cfg.B * cfg.N
        line = {"mode": "sweep", "metric": METRIC, "value": tokens / (attn_cold + acc_cold), "unit": UNIT,
                "n_gpus": 1, "steps": reps, "warmup": 3, "higher_is_better": True, "dtype": "bf16",
                "data": "synthetic",
                "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                           "L": cfg.L, "V": cfg.V, "depth": cfg.depth, "R": cfg.N * cfg.G,
                           "l2": "cold = a 504 MB buffer written between calls; warm = one resident set, CUDA-graph replay",
                           "num_splits": gsd.gsd_verify_attn_num_splits(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax)},
                "attn_us_cold": attn_cold * 1e6, "attn_us_warm": attn_warm * 1e6,
                "accept_us_cold": acc_cold * 1e6, "accept_us_warm": acc_warm * 1e6,
                "accept_frac_of_hbm_cold": accept_bytes / acc_cold / 1e9 / peaks["hbm_gbs"],
                "accept_frac_of_hbm_warm": accept_bytes / acc_warm / 1e9 / peaks["hbm_gbs"],
                "roofline": roof}
        print(json.dumps(line), flush=True)
        del t, out, ws, ws_acc
        torch.cuda.empty_cache()


def run_ab_balanced(args):
    """gsd_verify_attn with its fixed plan (made on the host from Lmax) against the two plans made
    on the device from seq_lens (equal shares of key tiles per group of CTAs; a split count per
    sequence), cold.  70B layer shape: a uniform batch, lengths drawn uniformly from [256, 8192],
    one 16384-token context among short ones; 13B layer shape (one kv head per query head): its
    own lengths, and 16 sequences with one long context.  One JSON line per batch."""
    import paper_2407_16207_b200 as gsd
    from gsd_inputs.torch_io import attn_tensors
    gsd.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks, peak_src = load_peaks()
    base = gi.CONFIGS["llama70b"]
    flush = torch.empty(4 * L2_BYTES, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    reps = max(args.steps if args.steps_given else 20, 3)
    mha = gi.CONFIGS["llama13b"]
    cases = [(base, "uniform_L4096", base.L, None), (base, "ragged_L256_8192", (256, 8192), None),
             (base, "one_long_L16384", 16384, (256, 1024)),
             (mha, "llama13b", mha.L, None),
             (gi.VerifyConfig(**{**mha.__dict__, "B": 16, "N": 64}), "mha_B16_one_long_L8192", 8192, (128, 1024))]
    for shape, name, L, others in cases:
        cfg = gi.VerifyConfig(**{**shape.__dict__, "name": name, "L": L})
        inp = gi.make_inputs(cfg, accept=False)
        if others is not None:
            # every sequence but the first is cut back to a short context
            rng = np.random.default_rng(gi.seed_for(cfg, 1))
            inp["seq_lens"][1:] = rng.integers(others[0], others[1] + 1, size=cfg.B - 1, dtype=np.int32)
        t = attn_tensors(inp, dev)
        out = torch.empty_like(t["q"])
        Lmax = inp["Lmax"]
        times, outs = {}, {}
        for ns in (0, gsd.GSD_ATTN_SPLIT_BALANCED, gsd.GSD_ATTN_SPLIT_PER_SEQUENCE):
            need = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax, ns)
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)

            def attn():
                gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                                    t["ancestor_mask"], t["seq_lens"], out=out, workspace=ws, status=status,
                                    num_splits=ns)
            for _ in range(3):
                attn()
            torch.cuda.synchronize()
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(reps)]
            for i in range(reps):
                flush.fill_(i & 0xFF)
                ev[i][0].record(); attn(); ev[i][1].record()
            torch.cuda.synchronize()
            times[ns] = statistics.median(e[0].elapsed_time(e[1]) for e in ev) * 1e-3
            outs[ns] = out.float().clone()
        if int(status.item()) != 0:
            raise RuntimeError(f"device status {int(status.item()):#x} on {name}")
        flops, attn_bytes, _ = algorithmic_work(cfg, inp)
        fixed, bal, seq = times[0], times[gsd.GSD_ATTN_SPLIT_BALANCED], times[gsd.GSD_ATTN_SPLIT_PER_SEQUENCE]
        lens = inp["seq_lens"]
        line = {"mode": "ab_balanced", "n_gpus": 1, "steps": reps, "warmup": 3, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D,
                           "seq_lens": {"min": int(lens.min()), "max": int(lens.max()), "mean": float(lens.mean())},
                           "l2": "cold = a 504 MB buffer written between calls"},
                "attn_us_fixed_plan": fixed * 1e6, "attn_us_balanced_plan": bal * 1e6,
                "attn_us_per_sequence_plan": seq * 1e6, "fixed_over_balanced": fixed / bal,
                "fixed_over_per_sequence": fixed / seq,
                "max_abs_difference_of_outputs": max(float((outs[0] - outs[m]).abs().max().item())
                                                     for m in (gsd.GSD_ATTN_SPLIT_BALANCED, gsd.GSD_ATTN_SPLIT_PER_SEQUENCE)),
                "roofline_fixed": roofline_of(flops, attn_bytes, fixed, peaks, peak_src),
                "roofline_balanced": roofline_of(flops, attn_bytes, bal, peaks, peak_src),
                "roofline_per_sequence": roofline_of(flops, attn_bytes, seq, peaks, peak_src)}
        print(json.dumps(line), flush=True)
        del t, out, outs
        torch.cuda.empty_cache()


def run_ab_unmerge(args):
    """Verification of the token graph itself (a node merged from several branches attends to
    the union of its ancestors) against verification of the paper's unmerged tree (Sec. 5.4): on
    graphs grown on the device by gsd_draft_expand from seeded draft logits whose mass sits on a
    small, context-dependent set of tokens (so that tau-grams re-occur as in the paper's Fig. 3),
    with the paper's settings k = 4, tau = 2, theta_prob = 0.2, theta_sib = 0.3, six draft steps
    (the paper allows ten; six keep the graph under this library's 512 nodes).
    Prints one JSON line: node counts, attention time of both forms on the 70B layer shape, and
    how far the attention rows of the two forms are apart."""
    import paper_2407_16207_b200 as gsd
    from gsd_inputs.torch_io import i32_tensor
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B, V, Ncap, k, tau, steps = 8, 32000, 512, 4, 2, 6
    Hq, Hkv, D, L = 64, 8, 128, 4096
    hot = 48                                             # tokens that ever get mass
    gen = torch.Generator(device=dev)
    gen.manual_seed(2407)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    tokens = torch.zeros((B, Ncap), dtype=torch.int32, device=dev)
    tokens[:, 0] = torch.randint(0, hot, (B,), device=dev, generator=gen, dtype=torch.int32)
    parent = torch.full((B, Ncap), -1, dtype=torch.int32, device=dev)
    merge = torch.full((B, Ncap), -1, dtype=torch.int32, device=dev)
    leaf = torch.zeros((B, Ncap), dtype=torch.uint8, device=dev)
    prob = torch.zeros((B, Ncap), dtype=torch.float32, device=dev)
    num = torch.ones((B,), dtype=torch.int32, device=dev)
    frontier = torch.zeros((B, 1), dtype=torch.int32, device=dev)
    flen = torch.ones((B,), dtype=torch.int32, device=dev)
    # the draft distribution after a token t: mass on six tokens of the hot set chosen by t
    table = torch.randint(0, hot, (hot, 6), device=dev, generator=gen)
    lvl = torch.tensor([4.0, 3.9, 3.8, 3.0, 2.0, 1.0], device=dev)      # three children of a node pass theta_prob = 0.2
    for _ in range(steps):
        F = int(frontier.shape[1])
        tok_f = torch.gather(tokens, 1, frontier.clamp(min=0).long())            # [B,F] token of each frontier node
        lg = torch.full((B, F, V), -8.0, device=dev) + 0.3 * torch.randn((B, F, V), device=dev, generator=gen)
        lg.scatter_(2, table[tok_f.long() % hot], (lvl + 0.2 * torch.randn((B, F, 6), device=dev, generator=gen)))
        nf, nfl = gsd.gsd_draft_expand(lg, frontier, flen, tokens, parent, merge, leaf, prob, num, k=k, tau=tau,
                                       theta_prob=0.2, theta_sib=0.3, status=status)
        width = int(nfl.max().item())
        if width == 0:
            break
        frontier, flen = nf[:, :width].contiguous().clamp(min=0), nfl
    torch.cuda.synchronize()
    graph_full = bool(int(status.item()) & 0x80)          # the node capacity ended the growth
    status.zero_()
    n = num.cpu().numpy()
    par_h, mrg_h = parent.cpu().numpy(), merge.cpu().numpy()
    N = int(n.max())
    # parent lists of the verification DAG: a node also hangs under the nodes merged into its parent
    parents = []
    for b in range(B):
        into = {}
        for r in range(n[b]):
            if mrg_h[b, r] >= 0:
                into.setdefault(int(mrg_h[b, r]), []).append(r)
        ps = [[]]
        for x in range(1, n[b]):
            p = int(par_h[b, x])
            ps.append(sorted([p] + [r for r in into.get(p, []) if r < x]))
        parents.append(ps + [[] for _ in range(N - n[b])])
    ptr, idx = gi.parents_to_csr(parents)
    d_ptr, d_idx = i32_tensor(ptr, dev), i32_tensor(idx, dev)
    d_tok = tokens[:, :N].contiguous()
    mask = gsd.gsd_build_mask(d_ptr, d_idx)
    q = torch.randn((B, N, Hq, D), device=dev, generator=gen).to(torch.bfloat16)
    dk = torch.randn((B, N, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    dv = torch.randn((B, N, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    kc = torch.randn((B, L, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    vc = torch.randn((B, L, Hkv, D), device=dev, generator=gen).to(torch.bfloat16)
    sl = torch.full((B,), L, dtype=torch.int32, device=dev)
    out_g = torch.empty_like(q)
    t_graph = timed_calls(lambda i: gsd.gsd_verify_attn(q, kc, vc, dk, dv, mask, sl, out=out_g, status=status))
    # the unmerged tree (at most Ncap nodes, at most `steps` edges deep), its single-parent lists and mask
    _, _, _, cnt_all = gsd.gsd_unmerge_tree(d_tok, d_ptr, d_idx, Ucap=1 << 16, max_depth=steps, status=status)
    tree_nodes_all = cnt_all.cpu().numpy()                 # the whole tree, for its size
    status.zero_()
    # the attention call takes at most 512 nodes: the first 512 of the level order are timed
    tt, tp, ts, cnt = gsd.gsd_unmerge_tree(d_tok, d_ptr, d_idx, Ucap=Ncap, max_depth=steps, status=status)
    torch.cuda.synchronize()
    full = bool(int(status.item()) & 0x200)
    status.zero_()
    cnt_h, tp_h = cnt.cpu().numpy(), tp.cpu().numpy()
    U = int(cnt_h.max())
    tparents = [[[] if (u == 0 or u >= cnt_h[b]) else [int(tp_h[b, u])] for u in range(U)] for b in range(B)]
    tptr, tidx = gi.parents_to_csr(tparents)
    tmask = gsd.gsd_build_mask(i32_tensor(tptr, dev), i32_tensor(tidx, dev))
    src = ts[:, :U].clamp(min=0).long()
    take = lambda x: torch.gather(x, 1, src.view(B, U, 1, 1).expand(-1, -1, x.shape[2], x.shape[3])).contiguous()
    q_t, dk_t, dv_t = take(q), take(dk), take(dv)
    out_t = torch.empty_like(q_t)
    t_tree = timed_calls(lambda i: gsd.gsd_verify_attn(q_t, kc, vc, dk_t, dv_t, tmask, sl, out=out_t, status=status))
    # rows of the graph form against the rows of their tree copies
    diff = (out_t.float() - take(out_g).float()).abs()
    valid = (torch.arange(U, device=dev)[None, :] < cnt[:, None])
    per_node = diff.amax(dim=(2, 3))[valid]
    line = {"mode": "ab_unmerge", "sequences": B, "draft_steps": steps, "k": k, "tau": tau,
            "graph_nodes_mean": float(n.mean()), "graph_nodes_max": N,
            "merged_nodes_mean": float((mrg_h >= 0).sum() / B), "graph_capacity_reached": graph_full,
            "tree_nodes_mean": float(tree_nodes_all.mean()), "tree_nodes_max": int(tree_nodes_all.max()),
            "tree_nodes_timed_mean": float(cnt_h.mean()), "tree_truncated_to_512_for_timing": full,
            "attn_us_graph": t_graph, "attn_us_tree": t_tree,
            "rows_graph": int(n.sum()) * Hq, "rows_tree": int(cnt_h.sum()) * Hq,
            "tree_copies_whose_row_differs": float((per_node > 1e-3).float().mean().item()),
            "max_abs_difference": float(per_node.max().item()), "mean_abs_difference": float(diff[valid].mean().item()),
            "shape": {"Hq": Hq, "Hkv": Hkv, "D": D, "L": L, "V": V}}
    print(json.dumps(line), flush=True)


def timed_calls(fn, before=None, n=20, warm=3):
    """Median CUDA-event time in microseconds of `fn(i)` over n calls after `warm` untimed ones;
    `before(i)` runs ahead of each call, outside its pair of events."""
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for i in range(n + warm):
        if before:
            before(i)
        if i >= warm:
            ev[i - warm][0].record()
        fn(i)
        if i >= warm:
            ev[i - warm][1].record()
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="llama70b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 mma.sync, 2 tcgen05")
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-baseline", default="auto", choices=["auto", "full", "sample", "off"],
                    help="auto: the whole step on the named configurations, a sample on sweep points")
    ap.add_argument("--sweep", action="store_true", help="one JSON line per point of the 70B-shaped sweep")
    ap.add_argument("--points", default="", help="with --sweep: comma-separated workload names")
    ap.add_argument("--ab-balanced", action="store_true",
                    help="fixed plan against balanced plan of gsd_verify_attn on uniform and ragged batches")
    ap.add_argument("--ab-unmerge", action="store_true",
                    help="graph-direct against unmerged-tree verification on grown graphs; one JSON line")
    args = ap.parse_args()
    args.steps_given = args.steps is not None
    if args.steps is None:
        args.steps = 6000
    if args.sweep:
        run_sweep(args)
        return
    if args.ab_balanced:
        run_ab_balanced(args)
        return
    if args.ab_unmerge:
        run_ab_unmerge(args)
        return
    cfg = config_by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import paper_2407_16207_b200 as gsd
    from gsd_inputs.torch_io import accept_tensors, attn_tensors
    gsd.lib()  # fail loudly if the CUDA library is missing
    rank, world, local, dist = dist_setup(args.gpus)
    dev = torch.device("cuda", local)

    # inputs: independent sets, rotated, so that every step reads more than the L2 holds
    # (126 MB) of data it has not just touched
    probe = gi.make_inputs(cfg, gi.seed_for(cfg, 10 * rank))
    set_bytes = sum(v.nbytes for v in probe.values() if isinstance(v, np.ndarray))
    NSETS = int(min(16, max(2, -(-3 * L2_BYTES // set_bytes))))
    host_sets = [probe] + [gi.make_inputs(cfg, gi.seed_for(cfg, 10 * rank + s)) for s in range(1, NSETS)]
    # ragged workloads draw their lengths per seed: every set's cache is padded (with rows no
    # sequence can see) to the longest padded length, so that one call shape serves all sets
    Lmax = max(h["Lmax"] for h in host_sets)
    for h in host_sets:
        if h["Lmax"] < Lmax:
            for key in ("k_cache", "v_cache"):
                old_c = h[key]
                pad = np.full((old_c.shape[0], Lmax - old_c.shape[1]) + old_c.shape[2:], 0x7E00, dtype=np.uint16)
                h[key] = np.concatenate([old_c, pad], axis=1)
            h["Lmax"] = Lmax
    sets = []
    for inp in host_sets:
        t = {**attn_tensors(inp, dev), **accept_tensors(inp, dev)}
        t["out"] = torch.empty_like(t["q"])
        sets.append(t)
    ws_bytes = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax,
                                                   args.num_splits, args.kernel)
    ws_attn = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
    ws_acc = torch.empty(gsd.gsd_accept_workspace_bytes(cfg.B, cfg.N), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    acc_out = (torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=dev),
               torch.empty((cfg.B,), dtype=torch.int32, device=dev),
               torch.empty((cfg.B, cfg.N), dtype=torch.int32, device=dev))
    splits = gsd.gsd_verify_attn_num_splits(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax,
                                            args.num_splits, args.kernel)

    def step(i, ev=None):
        t = sets[i % NSETS]
        if ev:
            ev[0].record()
        gsd.gsd_verify_attn(t["q"], t["k_cache"], t["v_cache"], t["draft_k"], t["draft_v"],
                            t["ancestor_mask"], t["seq_lens"], out=t["out"], kernel=args.kernel,
                            num_splits=args.num_splits, workspace=ws_attn, status=status)
        if ev:
            ev[1].record()
        gsd.gsd_accept(t["logits"], t["draft_tokens"], t["parent_ptr"], t["parent_idx"],
                       workspace=ws_acc, status=status, out=acc_out)
        if ev:
            ev[2].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    if sampler:
        sampler.start()
    e_begin.record()
    for i in range(args.steps):
        step(i, events[i])
    e_end.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    total_ms = e_begin.elapsed_time(e_end)
    attn_ms = [ev[0].elapsed_time(ev[1]) for ev in events]
    acc_ms = [ev[1].elapsed_time(ev[2]) for ev in events]
    if int(status.item()) != 0:
        raise RuntimeError(f"device status {int(status.item()):#x}")
    tokens = cfg.B * cfg.N
    agg = aggregate_over_ranks(total_ms / args.steps, tokens, world, dist, dev)
    ms_per_step, value = agg["ms_per_step"], agg["value"]
    total_ms = ms_per_step * args.steps

    # ---- side timings on rank 0, each call between its own CUDA events; none is part of `value`
    commit_us = sampled_us = draft_us = draft_us_big = None
    sampled_bytes = draft_bytes = draft_bytes_big = 0.0
    if rank == 0:
        # the cache update that follows the step (gsd_commit_kv) on a cache with head room
        t0s = sets[0]
        grow = cfg.depth + 1
        pad = torch.zeros((cfg.B, grow, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device=dev)
        kc2 = torch.cat([t0s["k_cache"], pad], dim=1).contiguous()
        vc2 = torch.cat([t0s["v_cache"], pad], dim=1).contiguous()
        sl0 = t0s["seq_lens"].clone()
        sl2 = sl0.clone()

        def commit(i):
            gsd.gsd_commit_kv(kc2, vc2, t0s["draft_k"], t0s["draft_v"], acc_out[2], acc_out[1], sl2, status=status)
        commit_us = timed_calls(commit, before=lambda i: sl2.copy_(sl0))
        del kc2, vc2, pad

        # non-deterministic verification (gsd_accept_sampled): the rotated logits as the target's,
        # the next set's logits as the draft model's (one row per sequence is read for the residual)
        gen = torch.Generator(device=dev)
        gen.manual_seed(7)
        dq = torch.rand((cfg.B, cfg.N), device=dev, generator=gen) * 0.5 + 0.01
        ua = torch.rand((cfg.B, cfg.N), device=dev, generator=gen)
        usm = torch.rand((cfg.B,), device=dev, generator=gen)
        ws_s = torch.empty(gsd.gsd_accept_sampled_workspace_bytes(cfg.B, cfg.N), dtype=torch.uint8, device=dev)

        acc_out_s = tuple(torch.empty_like(x) for x in acc_out)

        def sampled(i):
            ts, td = sets[i % NSETS], sets[(i + 1) % NSETS]
            gsd.gsd_accept_sampled(ts["logits"], ts["draft_tokens"], ts["parent_ptr"], ts["parent_idx"], dq, ua, usm,
                                   draft_logits=td["logits"], workspace=ws_s, status=status, out=acc_out_s)
        sampled_us = timed_calls(sampled)
        sampled_bytes = 4.0 * cfg.V * (cfg.B * cfg.N + cfg.B)

        # one growth step of the draft token graph (gsd_draft_expand): 64 frontier rows per
        # sequence of random draft logits over the same vocabulary, on a graph of 104 earlier nodes,
        # k = 4; once with the workload's batch and once with 32 sequences (262 MB of draft logits)
        def time_draft(Bd):
            gen.manual_seed(11)
            Fr, Ncap, n_old, k = 64, 512, 104, 4
            dl = [torch.randn((Bd, Fr, cfg.V), device=dev, generator=gen) * 3 for _ in range(2)]
            g_tok = torch.randint(0, cfg.V, (Bd, Ncap), device=dev, generator=gen, dtype=torch.int32)
            g_par = (torch.arange(Ncap, device=dev, dtype=torch.int32) - 1).clamp(min=0).repeat(Bd, 1).contiguous()
            g_par[:, 0] = -1
            g_mrg = torch.full((Bd, Ncap), -1, dtype=torch.int32, device=dev)
            g_leaf = torch.zeros((Bd, Ncap), dtype=torch.uint8, device=dev)
            g_prob = torch.zeros((Bd, Ncap), dtype=torch.float32, device=dev)
            n_ref = torch.full((Bd,), n_old, dtype=torch.int32, device=dev)
            g_n = n_ref.clone()
            fr = (torch.arange(Fr, device=dev, dtype=torch.int32) % n_old).repeat(Bd, 1).contiguous()
            fl = torch.full((Bd,), Fr, dtype=torch.int32, device=dev)
            nf = (torch.empty((Bd, Fr * k), dtype=torch.int32, device=dev), torch.empty((Bd,), dtype=torch.int32, device=dev))
            ws_d = torch.empty(Bd * Fr * 8 * 8 + 256, dtype=torch.uint8, device=dev)

            def draft(i):
                gsd.gsd_draft_expand(dl[i % 2], fr, fl, g_tok, g_par, g_mrg, g_leaf, g_prob, g_n, k=k, tau=2,
                                     theta_prob=0.01, theta_sib=0.1, status=status, workspace=ws_d, out=nf)
            us = timed_calls(draft, before=lambda i: g_n.copy_(n_ref))
            return us, 4.0 * Bd * Fr * cfg.V
        draft_us, draft_bytes = time_draft(cfg.B)
        draft_us_big, draft_bytes_big = time_draft(32)

    # ---- end to end through the host-buffer C-ABI call (pinned host tensors)
    e2e = None
    if args.e2e_steps > 0:
        h = {**attn_tensors(host_sets[0], "cpu"), **accept_tensors(host_sets[0], "cpu")}
        h = {k: v.pin_memory() for k, v in h.items()}
        Ecap = h["parent_idx"].shape[1]
        nbytes = gsd.gsd_verify_step_host_arena_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D, Lmax,
                                                      cfg.V, Ecap, cfg.N, args.num_splits, args.kernel)
        arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        h_out = torch.empty_like(h["q"]).pin_memory()
        h_acc = (torch.empty((cfg.B, cfg.N), dtype=torch.int32).pin_memory(),
                 torch.empty((cfg.B,), dtype=torch.int32).pin_memory(),
                 torch.empty((cfg.B, cfg.N), dtype=torch.int32).pin_memory())

        def host_step():
            return gsd.gsd_verify_step_host(
                h["q"], h["k_cache"], h["v_cache"], h["draft_k"], h["draft_v"], h["ancestor_mask"],
                h["seq_lens"], h["logits"], h["draft_tokens"], h["parent_ptr"], h["parent_idx"], arena,
                out=h_out, accepted=h_acc, kernel=args.kernel, num_splits=args.num_splits)

        for _ in range(2):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
        torch.cuda.synchronize()
        t_e2e = (time.perf_counter() - t0) / args.e2e_steps
        t_e2e = aggregate_over_ranks(t_e2e * 1e3, tokens, world, dist, dev)["ms_per_step"] * 1e-3
        h2d = sum(h[k].numel() * h[k].element_size() for k in h)
        d2h = h_out.numel() * 2 + sum(x.numel() * 4 for x in h_acc) + 4
        e2e = {"value": world * tokens / t_e2e, "unit": UNIT, "ms_per_step": t_e2e * 1e3,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        del arena

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    flops, attn_bytes, accept_bytes = algorithmic_work(cfg, host_sets[0])
    attn_med = statistics.median(attn_ms) * 1e-3
    attn_mean = sum(attn_ms) / len(attn_ms) * 1e-3
    acc_mean = sum(acc_ms) / len(acc_ms) * 1e-3
    roof = roofline_of(flops, attn_bytes, attn_mean, peaks, peak_src)
    roof["kernel"] = "gsd_verify_attn" + (" (split pass + merge pass)" if splits > 1 else "")
    if args.kernel in (0, 2) and args.num_splits == 0:
        # recorded only for workloads whose capture ran the tcgen05 kernel under the automatic choice
        roof["traffic"] = recorded_traffic("attn_tc_kernel", cfg.name)
    roof["launch_us_mean"] = attn_mean * 1e6
    roof["launch_us_median"] = attn_med * 1e6
    if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        # the same time scaled to the maximum SM clock (clock cycles are what the kernel costs)
        roof["launch_us_mean_at_max_clock"] = attn_mean * 1e6 * clocks["sm_mhz"] / clocks["sm_max_mhz"]

    cpu = None
    mode = args.cpu_baseline
    if mode == "auto":
        mode = "full" if cfg.name in gi.CONFIGS else "sample"
    if mode != "off" and world == 1:
        total_rows = cfg.B * cfg.N * cfg.Hq
        cpu = cpu_oracle_time(cfg, host_sets[0], total_rows if mode == "full" else 16384, 0)

    hbm = peaks["hbm_gbs"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv,
                   "D": cfg.D, "L": cfg.L, "V": cfg.V, "depth": cfg.depth,
                   "l2": (f"{NSETS} input sets of {set_bytes / 1e6:.0f} MB rotated"
                          + ("; together larger than L2" if NSETS * set_bytes > 2 * L2_BYTES else
                             "; together NOT larger than L2 (L2-warm numbers)")),
                   "replicas": world, "attn_kernel": args.kernel, "num_splits": splits},
        "attn_us": attn_mean * 1e6, "accept_us": acc_mean * 1e6, "commit_kv_us": commit_us,
        "accept_sampled_us": sampled_us, "draft_expand_us": draft_us,
        "attn_tokens_per_s": tokens / attn_mean,
        "accept_gbs": accept_bytes / acc_mean / 1e9,
        "accept_frac_of_hbm": accept_bytes / acc_mean / 1e9 / hbm,
        "accept_sampled_frac_of_hbm": (sampled_bytes / (sampled_us * 1e-6) / 1e9 / hbm) if sampled_us else None,
        "draft_expand_frac_of_hbm": (draft_bytes / (draft_us * 1e-6) / 1e9 / hbm) if draft_us else None,
        "draft_expand_262mb_us": draft_us_big,
        "draft_expand_262mb_frac_of_hbm": (draft_bytes_big / (draft_us_big * 1e-6) / 1e9 / hbm) if draft_us_big else None,
        "roofline": roof, "cpu_baseline": cpu, "e2e": e2e,
        # per step: the attention kernel (+ its merge pass when key ranges are cut), the scratch
        # clear of gsd_accept and the accept kernel
        "gpu_launches": args.steps * ((2 if splits > 1 else 1) + 2),
        "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
