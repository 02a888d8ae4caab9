#!/usr/bin/env python
"""Benchmark of the GSD verification step (gsd_verify_attn + gsd_accept) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama70b] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic LLaMA-2-shaped input:
DAG-masked attention of all draft nodes, then vocabulary argmax and longest accepted path.
Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent replica of the
workload (the path has no cross-GPU exchange), timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import gsd_inputs as gi  # noqa: E402

METRIC = "draft_tokens_verified_per_s_per_attn_layer"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


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
            self._stop.wait(0.02)

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


def cpu_oracle_sample(cfg, inp, budget_rows: int, accept_seqs: int = 0):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: `budget_rows`
    random attention rows plus the acceptance step of `accept_seqs` sequences (0 = all).
    Returns (tokens/s extrapolated to the whole step, threads, description)."""
    import oracle
    rng = np.random.default_rng(0)
    total_rows = cfg.B * cfg.N * cfg.Hq
    n = min(budget_rows, total_rows)
    rows = np.stack([rng.integers(cfg.B, size=n), rng.integers(cfg.N, size=n),
                     rng.integers(cfg.Hq, size=n)], axis=1).astype(np.int32)
    t0 = time.perf_counter()
    oracle.attn_rows(inp["q"], inp["k_cache"], inp["v_cache"], inp["draft_k"], inp["draft_v"],
                     inp["ancestor_mask"], inp["seq_lens"], rows)
    t_attn = time.perf_counter() - t0
    nb = cfg.B if accept_seqs <= 0 else min(accept_seqs, cfg.B)
    t0 = time.perf_counter()
    oracle.accept(inp["logits"][:nb], inp["draft_tokens"][:nb], inp["parent_ptr"][:nb], inp["parent_idx"][:nb])
    t_acc = (time.perf_counter() - t0) * (cfg.B / nb)
    t_step = t_attn * (total_rows / n) + t_acc
    desc = (f"{n} of {total_rows} attention rows (random (b,n,h), {t_attn:.3f} s, scaled to all rows) "
            f"+ acceptance of {nb} of {cfg.B} sequences ({t_acc:.3f} s scaled to all)")
    return cfg.B * cfg.N / t_step, oracle.threads(), desc


def run_reference(args, cfg):
    """The reference arm: the CPU oracle, timed on the host cores.  Each of the K steps is a
    bounded sample of the workload, sized so that the whole run takes about a minute whatever K is."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = gi.make_inputs(cfg)
    total_rows = cfg.B * cfg.N * cfg.Hq
    n_steps = args.warmup + args.steps
    # ~2e5 rows/min on 16 threads at this size: spread ~40000 rows over the run, at least 16 per step
    rows_per_step = int(min(total_rows, max(16, 40000 // max(1, n_steps))))
    accept_seqs = 0 if n_steps <= 50 else 1
    vals = []
    desc, threads = "", 1
    for i in range(n_steps):
        v, threads, desc = cpu_oracle_sample(cfg, inp, rows_per_step, accept_seqs)
        if i >= args.warmup:
            vals.append(v)
    value = cfg.B * cfg.N * len(vals) / sum(cfg.B * cfg.N / v for v in vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * cfg.B * cfg.N / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv,
                       "D": cfg.D, "L": cfg.L, "V": cfg.V},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": "per step: " + desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="llama70b", choices=sorted(gi.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 mma.sync, 2 tcgen05")
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-rows", type=int, default=16384,
                    help="attention rows in the CPU-oracle sample (0 = skip the CPU baseline)")
    args = ap.parse_args()
    cfg = gi.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import paper_2407_16207_b200 as gsd
    from gpu_util import accept_tensors, attn_tensors
    gsd.lib()  # fail loudly if the CUDA library is missing
    rank, world, local, dist = dist_setup(args.gpus)
    dev = torch.device("cuda", local)

    # inputs: two independent sets, rotated, so that every step reads ~0.5 GB it has not just
    # touched (more than the 126 MB L2)
    NSETS = 2
    host_sets = [gi.make_inputs(cfg, gi.seed_for(cfg, 10 * rank + s)) for s in range(NSETS)]
    sets = []
    for inp in host_sets:
        t = {**attn_tensors(inp, dev), **accept_tensors(inp, dev)}
        t["out"] = torch.empty_like(t["q"])
        sets.append(t)
    Lmax = host_sets[0]["Lmax"]
    ws_bytes = gsd.gsd_verify_attn_workspace_bytes(cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D,
                                                   max(h["Lmax"] for h in host_sets),
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

    # ---- the cache update that follows the step (gsd_commit_kv), timed on its own on a cache with
    # head room; it is not part of `value`
    commit_us = None
    if rank == 0:
        t0s = sets[0]
        grow = cfg.depth + 1
        kc2 = torch.cat([t0s["k_cache"], torch.zeros((cfg.B, grow, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device=dev)], dim=1).contiguous()
        vc2 = torch.cat([t0s["v_cache"], torch.zeros((cfg.B, grow, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device=dev)], dim=1).contiguous()
        sl0 = t0s["seq_lens"].clone()
        sl2 = sl0.clone()
        ev_c = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for i in range(23):
            sl2.copy_(sl0)
            if i >= 3:
                ev_c[i - 3][0].record()
            gsd.gsd_commit_kv(kc2, vc2, t0s["draft_k"], t0s["draft_v"], acc_out[2], acc_out[1], sl2, status=status)
            if i >= 3:
                ev_c[i - 3][1].record()
        torch.cuda.synchronize()
        commit_us = statistics.median(a.elapsed_time(b) for a, b in ev_c) * 1e3
        del kc2, vc2

    # ---- non-deterministic verification (gsd_accept_sampled) on the same logits, timed on its
    # own with the two input sets rotated; it is not part of `value`
    sampled_us = None
    if rank == 0:
        gen = torch.Generator(device=dev)
        gen.manual_seed(7)
        dq = torch.rand((cfg.B, cfg.N), device=dev, generator=gen) * 0.5 + 0.01
        ua = torch.rand((cfg.B, cfg.N), device=dev, generator=gen)
        usm = torch.rand((cfg.B,), device=dev, generator=gen)
        ws_s = torch.empty(gsd.gsd_accept_sampled_workspace_bytes(cfg.B, cfg.N), dtype=torch.uint8, device=dev)
        ev_s = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for i in range(23):
            ts = sets[i % len(sets)]
            if i >= 3:
                ev_s[i - 3][0].record()
            gsd.gsd_accept_sampled(ts["logits"], ts["draft_tokens"], ts["parent_ptr"], ts["parent_idx"], dq, ua, usm,
                                   workspace=ws_s, status=status)
            if i >= 3:
                ev_s[i - 3][1].record()
        torch.cuda.synchronize()
        sampled_us = statistics.median(a.elapsed_time(b) for a, b in ev_s) * 1e3

    # ---- one growth step of the draft token graph (gsd_draft_expand): 64 frontier rows per
    # sequence of random draft logits over the same vocabulary, on a graph of 104 earlier nodes;
    # timed on its own, not part of `value`
    draft_us = None
    if rank == 0:
        gen = torch.Generator(device=dev)
        gen.manual_seed(11)
        Fr, Ncap, n_old = 64, 512, 104
        dl = [torch.randn((cfg.B, Fr, cfg.V), device=dev, generator=gen) * 3 for _ in range(2)]
        g_tok = torch.randint(0, cfg.V, (cfg.B, Ncap), device=dev, generator=gen, dtype=torch.int32)
        g_par = (torch.arange(Ncap, device=dev, dtype=torch.int32) - 1).clamp(min=0).repeat(cfg.B, 1).contiguous()
        g_par[:, 0] = -1
        g_mrg = torch.full((cfg.B, Ncap), -1, dtype=torch.int32, device=dev)
        g_leaf = torch.zeros((cfg.B, Ncap), dtype=torch.uint8, device=dev)
        g_prob = torch.zeros((cfg.B, Ncap), dtype=torch.float32, device=dev)
        n_ref = torch.full((cfg.B,), n_old, dtype=torch.int32, device=dev)
        g_n = n_ref.clone()
        fr = (torch.arange(Fr, device=dev, dtype=torch.int32) % n_old).repeat(cfg.B, 1).contiguous()
        fl = torch.full((cfg.B,), Fr, dtype=torch.int32, device=dev)
        ev_d = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for i in range(23):
            g_n.copy_(n_ref)
            if i >= 3:
                ev_d[i - 3][0].record()
            gsd.gsd_draft_expand(dl[i % 2], fr, fl, g_tok, g_par, g_mrg, g_leaf, g_prob, g_n, k=4, tau=2,
                                 theta_prob=0.01, theta_sib=0.1, status=status)
            if i >= 3:
                ev_d[i - 3][1].record()
        torch.cuda.synchronize()
        draft_us = statistics.median(a.elapsed_time(b) for a, b in ev_d) * 1e3
        del dl

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
    t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12)
    t_hbm = attn_bytes / (peaks["hbm_gbs"] * 1e9)
    sustained = total_ms >= 2000.0
    if t_tc >= t_hbm:
        peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
        achieved = flops / attn_mean / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": None,
                "peak_kind": f"{'sustained' if sustained else 'burst'} bf16, of {peak_src}",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_burst": achieved / peaks["bf16_tflops"],
                "frac_of_nominal_2250": achieved / 2250.0}
    else:
        peak = peaks["hbm_gbs"]
        achieved = attn_bytes / attn_mean / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": None, "peak_kind": f"copy bandwidth, of {peak_src}",
                "frac_of_nominal_8000": achieved / 8000.0}
    # DRAM bytes of one launch of the dominant kernel from the committed ncu capture
    # (profiles/attn_tcgen05_llama70b.md); only valid for that kernel on that workload
    if cfg.name == "llama70b" and args.kernel in (0, 2) and args.num_splits == 0:
        roof["traffic"] = 197.7e6
    roof["kernel"] = "gsd_verify_attn" + (" (split pass + merge pass)" if splits > 1 else "")
    roof["algorithmic_flops"] = flops
    roof["algorithmic_bytes"] = attn_bytes
    roof["launch_us_mean"] = attn_mean * 1e6
    roof["launch_us_median"] = attn_med * 1e6

    cpu = None
    if args.cpu_rows > 0 and world == 1:
        v, threads, desc = cpu_oracle_sample(cfg, host_sets[0], args.cpu_rows)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "Hq": cfg.Hq, "Hkv": cfg.Hkv,
                   "D": cfg.D, "L": cfg.L, "V": cfg.V, "depth": cfg.depth,
                   "l2": "two input sets rotated; each step reads more than the L2 size",
                   "replicas": world, "attn_kernel": args.kernel, "num_splits": splits},
        "attn_us": attn_mean * 1e6, "accept_us": acc_mean * 1e6, "commit_kv_us": commit_us, "accept_sampled_us": sampled_us, "draft_expand_us": draft_us,
        "attn_tokens_per_s": tokens / attn_mean,
        "accept_gbs": accept_bytes / acc_mean / 1e9,
        "accept_frac_of_hbm": accept_bytes / acc_mean / 1e9 / peaks["hbm_gbs"],
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
