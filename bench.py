#!/usr/bin/env python
"""Benchmark of the encrypted linear layer: ms per decode token on one B200 (or N independent
replicas, one process per GPU), with the roofline of the dominant kernels and the CPU oracle
timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload qwen3_step@budget=60] [--impl reference]

A step = one decode token's worth of the workload: the encrypted product and its rescale
(bf_linear_rescaled: bf_linear + bf_rescale as one call) for every linear layer of the workload, cached encoded weights streamed from HBM (49 GB per step for the Qwen3-0.6B-shaped
default, 352 MB for the single GPT-2 projection: always larger than L2, so consecutive steps cannot
be served from cache).  The other configurations are timed after the main one and reported under
"other_workloads", each with its own rooflines.  Inputs are seeded and synthetic.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "encrypted linear-layer ms per decode token"
UNIT = "ms"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) relative to the algorithmic bytes of the same launches,
# from ncu captures summarised under profiles/.  The headline workload is too large for a multi-pass capture (37.6 GB on
# the device), so the figures come from one GPT-2 layer under the same plan (same kernels, same call shapes), whose
# traffic grows in proportion to the streamed bytes; `traffic` in the line = this ratio x the algorithmic bytes of a launch.
NCU_TRAFFIC_RATIO = {
    "mac": 1.32,                  # eight captured launches (four calls): 1417 MB for 1074 MB of cached words (rotated inputs, outputs)
    "key_inner_product": 1.40,    # eight captured launches: 1352 MB for 33 distinct keys of 29.36 MB (digit sets, outputs)
}
# (ncu flushes the caches before every captured launch: rotated inputs and digit sets that a step finds in L2 count as
# DRAM traffic in these ratios)
# Executed warp instructions per butterfly by pipe, from the same captures (profiles/gpt2_layer_headline_plan_kernels_ncu.md),
# to set beside the modelled 8 / 12 / 10 operations: the large fp64-path batches of each direction.
NCU_PIPE_INSTR = {
    "ntt_forward": {"all": 24.7, "fp64": 8.3, "alu": 6.3, "fma_integer": 5.4, "lsu": 2.4,
                    "from": "hoisted ModUp of three inputs (147 transforms: six primes on the 8-operation fp64 path, one "
                            "on the 12-operation one, one on the 60-bit integer path), both passes"},
    "ntt_inverse": {"all": 21.0, "fp64": 10.3, "alu": 3.9, "fma_integer": 2.0, "lsu": 2.3,
                    "from": "c1 of 3 giant rotations x 7 primes, both passes (an earlier capture of the same kernels)"},
}


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        super().__init__(daemon=True)
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def run(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                self.lines.append((time.time(), line.strip()))
        except Exception:
            pass

    def stop(self):
        if self.proc:
            self.proc.terminate()

    def summary(self, t0: float, t1: float) -> dict:
        sm, smax, reasons, power = [], [], set(), []
        for ts, line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7 or not (t0 <= ts <= t1 + 0.06):
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


DEFAULT_LANES = 2       # the library's default number of concurrent key-switch chains
MIN_REGION_S = 0.5      # every timed region lasts at least this long (steps are repeated inside it)

# Workload specifications: "<workload>[@option[,option...]]".  Options: budget=<GB> (cache budget, so that
# overflow layers take the on-the-fly path), on_the_fly (budget of one byte: nothing is cached), compact
# (compact cache format), fold (in-ciphertext fold of the tau partial sums), complex (two output row blocks per
# plaintext, in the real and imaginary parts of the slots), per_output (one division by the special prime per
# output ciphertext instead of one per giant rotation), double_hoist (baby-step rotations kept in the extended basis,
# one division per inner sum), coeff64 / coeff32 (cached weights kept as rounded integer coefficients and transformed
# on every call).
# The headline is the largest single-GPU configuration under the fastest plan variant that is parity-tested; the same
# step under the plain plan, and the other configurations under both, follow as extras.
BEST = "complex,per_output,double_hoist"
DEFAULT_WORKLOAD = "qwen3_step@budget=60," + BEST
DEFAULT_EXTRA = ",".join([
    "qwen3_step@budget=60", "qwen3_step@budget=40.5", "qwen3_step@budget=40.5,compact", "qwen3_step@coeff32," + BEST,
    "gpt2_qkv", "gpt2_qkv@" + BEST, "gpt2_step", "gpt2_step@" + BEST,
    "llama3_layer", "llama3_layer@" + BEST, "llama3_layer@on_the_fly", "llama3_layer@on_the_fly," + BEST, "tiny"])


def parse_spec(spec: str):
    name, _, opts = spec.partition("@")
    kw = {}
    for o in filter(None, opts.split(",")):
        if o.startswith("budget="):
            kw["cache_budget_bytes"] = int(float(o[7:]) * 10 ** 9)
        elif o == "on_the_fly":
            kw["cache_budget_bytes"] = 1
        elif o == "compact":
            kw["compact_cache"] = True
        elif o == "fold":
            kw["fold_in_ciphertext"] = True
        elif o == "complex":
            kw["pack"] = "complex"
        elif o == "per_output":
            kw["moddown"] = "per_output"
        elif o == "double_hoist":
            kw["hoist"] = "double"
        elif o in ("coeff64", "coeff32"):
            kw["coef_bits"] = int(o[5:])
        elif o.startswith("lanes="):
            kw["lanes"] = int(o[6:])
        else:
            raise ValueError(f"unknown workload option {o!r}")
    return name, kw


def split_specs(text: str):
    """Comma-separated specs; an item without a workload name in front is an option of the previous spec."""
    from paper_2606_17421_b200 import workloads as wl
    out = []
    for item in filter(None, text.split(",")):
        if item.split("@")[0] in wl.WORKLOADS:
            out.append(item)
        else:
            out[-1] += ("," if "@" in out[-1] else "@") + item
    return out


def transform_counts(runner) -> dict:
    """Transforms one step launches, by direction and by arithmetic path.  Moduli below 2^41 run in
    fp64 with 8 fp64 operations per butterfly (signed lazy values), moduli from 2^41 up to 2^50 in fp64
    with a conditional subtraction and offsets (12 operations), the 60-bit special prime in integers
    (at least 10 32-bit multiply-adds per butterfly)."""
    import math
    r, N = runner.r, runner.N
    per = (N // 2) * int(math.log2(N))
    moduli = list(runner.primes) + [runner.P]
    cost = [8 if q < (1 << 41) else 12 if q < (1 << 50) else 10 for q in moduli]
    fp = [q < (1 << 50) for q in moduli]
    fwd = [0] * (r + 1)
    inv = [0] * (r + 1)
    for e in runner.layers:
        n_in, n_out, b, g = e["n_in"], e["n_out"], e["b"], e["g"]
        n_giant = (g - 1) * n_out
        sets = (n_in if b > 1 else 0) + n_giant            # ModUp digit sets
        rots = n_in * (b - 1) + n_giant                    # key switches
        # divisions by P: one per rotation and component, or (per_output) one per baby rotation and per output
        n_baby_lift = 2 * n_out * g if runner.plan.hoist == "double" else 2 * n_in * (b - 1)
        n_lift = n_baby_lift + 2 * (n_out if runner.plan.moddown == "per_output" and n_giant else n_giant)
        if runner.plan.hoist == "double" and runner.plan.moddown == "per_output" and n_giant:
            # inner sums stay in the extended basis: no lifted P-residue is transformed; the giant steps' ModUp divides in
            # its first load (and transforms each digit in its own prime too); the outputs are assembled by one inverse
            # transform per residue, g + 3 of them modulo P per output
            baby_sets = n_in if b > 1 else 0
            for i in range(r):
                fwd[i] += 2 * n_in + baby_sets * (r - 1) + n_giant * r
                inv[i] += n_giant + 2 * n_out
            fwd[r] += sets * r
            inv[r] += n_giant + n_out * (g + 3)
        else:
            for i in range(r):
                fwd[i] += 2 * n_in + sets * (r - 1) + n_lift   # inputs; digits of the other primes; lifted P-residues
                inv[i] += n_giant + 2 * n_out                  # c1 of the giant-step inputs; outputs
            fwd[r] += sets * r
            inv[r] += n_lift                                   # P-residues of the inner products
        if runner.transforms_weights_per_call(e):          # on the fly or kept as coefficients: every diagonal is transformed on each call
            n_diag = n_in * n_out * b * g
            for i in range(r + (1 if runner.plan.hoist == "double" else 0)):
                fwd[i] += n_diag
    def summary(cnt):
        return {"polys": sum(cnt), "fp64_polys": sum(c for c, f in zip(cnt, fp) if f),
                "fp64_ops": sum(c * k for c, k, f in zip(cnt, cost, fp) if f),
                "int_ops": sum(c * k for c, k, f in zip(cnt, cost, fp) if not f)}
    return {"fwd": summary(fwd), "inv": summary(inv), "per_poly": per}


class Measurement:
    """Times one workload on the current device: K steps (repeated so that the region lasts at least
    MIN_REGION_S) with the default launch configuration, then the same steps with an event pair around
    every launch and the key-switch chains serialised, from which the per-kernel rooflines follow."""

    def __init__(self, spec: str, seed: int = 0, device: str = "cuda:0", world: int = 1):
        from paper_2606_17421_b200.runner import WorkloadRunner
        self.spec = spec
        name, kw = parse_spec(spec)
        self.name = name
        self.world = world
        self.R = WorkloadRunner(name, seed=seed, device=device, **kw)

    def barrier(self):
        import torch
        import torch.distributed as dist
        torch.cuda.synchronize()
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(self, fn, count):
        """count calls of fn between two events on the runner's stream; (max-over-ranks ms, wall t0, wall t1)"""
        import torch
        from paper_2606_17421_b200.replicas import max_over_ranks
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        t0 = time.time()
        e0.record(self.R.stream)
        for _ in range(count):
            fn()
        e1.record(self.R.stream)
        self.barrier()
        t1 = time.time()
        return max_over_ranks(e0.elapsed_time(e1), device="cuda"), t0, t1

    def repeats_for(self, fn, steps):
        """How often a step is repeated inside the timed region so that it lasts MIN_REGION_S (same on all ranks)."""
        import math
        ms, _, _ = self.timed(fn, 1)
        return max(1, math.ceil(MIN_REGION_S * 1e3 / max(1e-3, ms * steps)))

    def run(self, steps: int, warmup: int, e2e: bool = False) -> dict:
        from paper_2606_17421_b200 import bifrost as bf
        R = self.R
        for _ in range(max(warmup, 3)):
            R.step()
        reps = self.repeats_for(R.step, steps)
        self.barrier()
        bf.bf_get_kernel_stats(R.ctx)   # reset launch counters
        ms_total, t0, t1 = self.timed(R.step, steps * reps)
        stats = bf.bf_get_kernel_stats(R.ctx)
        out = {"ms_per_step": ms_total / (steps * reps), "repeats_per_step": reps, "t0": t0, "t1": t1,
               "gpu_launches": sum(v[0] for v in stats.values()),
               "launches_per_step": sum(v[0] for v in stats.values()) / (steps * reps)}
        # per-kernel durations: an event pair around every launch, chains serialised (one lane) so that no other
        # kernel of the step runs beside the timed one
        k_steps = max(1, min(steps * reps, max(3, int(0.3 * steps * reps))))
        bf.bf_set_kernel_timing(R.ctx, True)
        bf.bf_set_lanes(R.ctx, 1)
        bf.bf_get_key_stream_bytes(R.ctx)
        self.timed(R.step, k_steps)
        out["kstats"] = bf.bf_get_kernel_stats(R.ctx)
        out["key_bytes"] = bf.bf_get_key_stream_bytes(R.ctx)
        out["k_steps"] = k_steps
        bf.bf_set_kernel_timing(R.ctx, False)
        bf.bf_set_lanes(R.ctx, DEFAULT_LANES)
        if e2e:
            # end to end through the host-buffer entry point (pinned host ciphertexts in and out)
            R.make_host_buffers()
            for _ in range(2):
                R.step_host()
            e_reps = self.repeats_for(R.step_host, 3)
            e_steps = 3 * e_reps
            e_total, _, _ = self.timed(R.step_host, e_steps)
            out["e2e_ms"] = e_total / e_steps
            out["e2e_steps"] = e_steps
        return out

    def rooflines(self, m: dict, hbm_peak: float, peak_kind: str, fma_rate: float, imad_rate: float) -> dict:
        R, kstats, K = self.R, m["kstats"], m["k_steps"]
        def traffic_of(kind, algorithmic_bytes):
            ratio = NCU_TRAFFIC_RATIO.get(kind)
            return round(ratio * algorithmic_bytes) if ratio and algorithmic_bytes else None
        counts = transform_counts(R)

        def avg_ms(cat):
            n, ms = kstats[cat]
            return (ms / n) if n else None, n / K

        rl = {}
        # weight-streaming multiply-accumulate: algorithmic bytes = every encoded word once
        mac_ms, mac_n = avg_ms("mac")
        if mac_ms:
            mac_bytes = R.total_pt_bytes() / max(1.0, mac_n)
            ach = mac_bytes / (mac_ms * 1e-3) / 1e9
            rl["mac"] = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s",
                         "frac": round(ach / hbm_peak, 4), "of": peak_kind, "traffic": traffic_of("mac", mac_bytes),
                         "launches_per_step": mac_n, "avg_ms": round(mac_ms, 5),
                         "bytes_per_launch": round(mac_bytes), "frac_of_nominal_8000": round(ach / 8000.0, 4)}
            if R.plan.hoist == "double":
                rl["mac"]["note"] = ("a call's two launches (ciphertext primes; the special prime beside it on a second "
                                     "stream) are timed as one span, the way they run; avg_ms = that span / 2")
        # key-switch inner product: algorithmic bytes = every distinct key of a launch once
        ki_ms, ki_n = avg_ms("key_inner_product")
        if ki_ms:
            distinct, per_rot = m["key_bytes"]
            n_launch = kstats["key_inner_product"][0]
            ach = distinct / n_launch / (ki_ms * 1e-3) / 1e9
            ach_rot = per_rot / n_launch / (ki_ms * 1e-3) / 1e9
            rl["key_inner_product"] = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s",
                                       "frac": round(ach / hbm_peak, 4), "of": peak_kind,
                                       "traffic": traffic_of("key_inner_product", distinct / n_launch),
                                       "launches_per_step": ki_n, "avg_ms": round(ki_ms, 5),
                                       "bytes_per_launch": round(distinct / n_launch),
                                       "achieved_counting_a_key_per_rotation": round(ach_rot, 1),
                                       "note": "bytes = the distinct keys of a launch, each once; the second figure "
                                               "counts a key once per rotation (repeats are L2 hits)"}
        # transforms: bound by the arithmetic pipes (fp64 for the ciphertext primes, integer multiply-add for the
        # special prime); the peak uses the two rates measured in this run
        for cats, key, label in ((("ntt_fwd_strided", "ntt_fwd_contig"), "fwd", "ntt_forward"),
                                 (("ntt_inv_contig", "ntt_inv_strided"), "inv", "ntt_inverse")):
            ms_step = sum(kstats[c][1] for c in cats) / K
            if ms_step > 0:
                info = counts[key]
                rate = info["polys"] * counts["per_poly"] / (ms_step * 1e-3)
                t_poly = (info["fp64_ops"] / fma_rate + info["int_ops"] / imad_rate) / max(1, info["polys"])
                peak = 1.0 / t_poly
                rl[label] = {"bound": "alu", "achieved": round(rate / 1e9, 1), "peak": round(peak / 1e9, 1),
                             "unit": "G butterflies/s", "frac": round(rate / peak, 4),
                             "of": (f"measured in this run: {fma_rate / 1e12:.2f} T fp64 multiply-adds/s and "
                                    f"{imad_rate / 1e12:.2f} T 32-bit integer multiply-adds/s over the GPU; modelled "
                                    "operations per butterfly: 8 fp64 below 2^41, 12 fp64 up to 2^50, 10 integer for the "
                                    "special prime"),
                             "pipe_instructions_per_butterfly_ncu": NCU_PIPE_INSTR.get(label),
                             "traffic": None, "ms_per_step": round(ms_step, 5),
                             "polys_per_step": info["polys"], "fp64_polys_per_step": info["fp64_polys"]}
        total_k_ms = sum(v[1] for v in kstats.values())
        shares = {k: round(v[1] / total_k_ms, 4) for k, v in kstats.items() if v[0]}
        return {"rooflines": rl, "kernel_time_share": shares,
                "kernel_ms_per_step": {k: round(v[1] / K, 4) for k, v in kstats.items() if v[0]}}

    def describe(self) -> dict:
        R = self.R
        h2d, d2h = R.host_bytes_per_step()
        whole_step = R.w.n_repeat > 1 or len(R.w.layers) > 1
        return {"layers": len(R.layers), "unit_of_work": "decode token (all linear layers)" if whole_step else "one projection call",
                "ring_N": R.N, "ct_primes": R.r,
                "plan": {"D": R.plan.D, "tau": R.plan.tau, "b": R.plan.b, "g": R.plan.g, "pack": R.plan.pack,
                         "moddown": R.plan.moddown, "hoist": R.plan.hoist,
                         "splits_per_call": {k: f"{b}x{g}" for k, (b, g) in R.splits.items()
                                             if (b, g) != (R.plan.b, R.plan.g)}},
                "ciphertexts_in": sum(e["n_in"] for e in R.layers), "ciphertexts_out": sum(e["n_out"] for e in R.layers),
                "boundary_bytes": h2d + d2h, "rotation_keys": len(R.rot_steps), "fallback_layers": R.n_fallback_layers(),
                "encoded_weight_bytes_cached": R.cached_pt_bytes(), "encoded_weight_bytes_total": R.total_pt_bytes(),
                "resident_weight_bytes": R.resident_bytes()}

    def close(self):
        import torch
        self.R.close()
        torch.cuda.empty_cache()


def measure_extra(spec: str, steps: int, peaks) -> dict:
    M = Measurement(spec)
    try:
        m = M.run(steps, 3)
        out = M.describe()
        key = "ms_per_token" if out["unit_of_work"].startswith("decode token") else "ms_per_call"
        out[key] = round(m["ms_per_step"], 4)
        out["repeats_per_step"] = m["repeats_per_step"]
        out["launches_per_step"] = m["launches_per_step"]
        out.update(M.rooflines(m, *peaks))
        return out
    finally:
        M.close()


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2606_17421_b200 import bifrost as bf
    from paper_2606_17421_b200.replicas import job_ms_per_token

    bf.load()   # fails loudly when the CUDA library is missing
    # every rank decodes its own token stream (independent problems: no data-path collective)
    M = Measurement(args.workload, seed=rank, device=f"cuda:{local}", world=world)
    R = M.R
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    m = M.run(args.steps, args.warmup, e2e=True)
    sampler.stop()
    clocks = sampler.summary(m["t0"], m["t1"])
    ms_per_step = m["ms_per_step"]

    if rank != 0:
        M.close()
        if world > 1:
            dist.destroy_process_group()
        return

    hbm_peak, peak_kind = read_peaks()
    imad_rate = bf.bf_measure_imad_rate(R.ctx)
    fma_rate = bf.bf_measure_fma64_rate(R.ctx)
    peaks = (hbm_peak, peak_kind, fma_rate, imad_rate)
    info = M.rooflines(m, *peaks)
    rooflines, shares = info["rooflines"], info["kernel_time_share"]
    dominant = max(shares, key=shares.get)
    dom_key = {"ntt_fwd_strided": "ntt_forward", "ntt_fwd_contig": "ntt_forward", "ntt_inv_contig": "ntt_inverse",
               "ntt_inv_strided": "ntt_inverse"}.get(dominant, dominant)
    roofline = dict(rooflines.get(dom_key, rooflines.get("mac", {})))
    roofline["kernel"] = dom_key

    desc = M.describe()
    h2d, d2h = R.host_bytes_per_step()
    sm_mhz = clocks.get("sm_mhz") or 1965.0
    line = {
        "metric": METRIC, "value": round(job_ms_per_token(ms_per_step, world), 5), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5),
        "repeats_per_step": m["repeats_per_step"],
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": args.workload, "unit_of_work": desc["unit_of_work"], "ring_N": R.N, "ct_primes": R.r,
                   "plan": desc["plan"], "layers": len(R.layers),
                   "encoded_weight_bytes_per_step": R.total_pt_bytes(),
                   "encoded_weight_bytes_cached": R.cached_pt_bytes(), "fallback_layers": R.n_fallback_layers(),
                   "l2": "inputs larger than L2: the encoded weights streamed each step exceed 126 MB",
                   "timed_region": f"{args.steps} steps x {m['repeats_per_step']} repeats, at least {MIN_REGION_S} s",
                   "multi_gpu": "replicas: every rank decodes its own token, no data-path collective"},
        "tokens_per_s": round(world * 1e3 / ms_per_step, 3),
        "clocks": clocks,
        "e2e": {"value": round(job_ms_per_token(m["e2e_ms"], world), 5), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": m["e2e_steps"]},
        "gpu_launches": m["gpu_launches"],
        "roofline": roofline,
        "rooflines": rooflines,
        "kernel_time_share": shares,
        "kernel_ms_per_step": info["kernel_ms_per_step"],
        "kernel_timing": "event pair around every launch with the key-switch chains serialised (1 lane); "
                         f"value and e2e are timed with {DEFAULT_LANES} concurrent chains and no per-launch events",
        "measured_rates": {"imad_per_sm_clk": round(imad_rate / 148 / (sm_mhz * 1e6), 2),
                           "fma64_per_sm_clk": round(fma_rate / 148 / (sm_mhz * 1e6), 2),
                           "imad_per_s": imad_rate, "fma64_per_s": fma_rate},
    }
    M.close()
    if world == 1 and args.extra:
        extras = {}
        for spec in split_specs(args.extra):
            name, _ = parse_spec(spec)
            steps = 200 if name in ("tiny", "gpt2_qkv", "gpt2_qkv_paper_params") or name.startswith("gemm1024") else 5
            extras[spec] = measure_extra(spec, steps, peaks)
        full, part = extras.get("qwen3_step@budget=60"), extras.get("qwen3_step@budget=40.5")
        if full and part:
            # 60 GB keeps every layer resident; 40.5 GB = 23/28 of the plain plan's encoded size reproduces the partially
            # cached regime (Sec. 6.1, table "FHE decode cost breakdown"): the overflow layers are encoded on every call
            part["fallback_share_of_step"] = round(1.0 - full["ms_per_token"] / part["ms_per_token"], 4)
        for tail in ("", "," + BEST):
            a, b = extras.get("llama3_layer" + ("@" + BEST if tail else "")), extras.get("llama3_layer@on_the_fly" + tail)
            if a and b:
                b["on_the_fly_over_cached"] = round(b["ms_per_token"] / a["ms_per_token"], 3)
        line["other_workloads"] = extras
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=20.0)
    elif world == 1:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# CPU oracle leg

class OracleSample:
    """The oracle on a bounded sample of the workload's first layer: all baby steps of `n_baby` of
    the b-1 rotations of one input ciphertext, and `n_groups` of the n_out*g (output block, giant
    step) groups; the step time is scaled to the whole layer by those counts, and to the whole
    workload by encoded-diagonal count."""

    def __init__(self, spec: str):
        import numpy as np
        from oracle import ckks
        from paper_2606_17421_b200 import workloads as wl
        self.np, self.ckks = np, ckks
        workload, kw = parse_spec(spec)
        w = wl.WORKLOADS[workload]
        ps = wl.PARAM_SETS[w.params]
        self.w = w
        self.par = ckks.Params(ps["N"], list(ps["primes"]), ps["special"], ps["scale"])
        self.plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, pack=kw.get("pack", w.plan.pack),
                              moddown=kw.get("moddown", w.plan.moddown), hoist=kw.get("hoist", w.plan.hoist))
        self.L = w.layers[0]
        self.W = wl.gen_weights(0, self.L.name, self.L.d_out, self.L.d_in)
        x = wl.gen_activation(0, self.L.name, self.L.d_in)
        self.s = ckks.keygen(self.par, 0)
        self.cts = ckks.encrypt_vector(self.par, self.plan, self.s, x, 0)
        self.keys = {}
        self.n_in = len(self.cts)
        self.n_out = self.plan.n_out(self.L.d_out)
        self.encoded = {}
        self.Xh = None

    def key_for(self, steps):
        ck = self.ckks
        g = ck.galois_element(steps, self.par.N)
        if steps % self.par.n and g not in self.keys:
            self.keys[g] = ck.galois_key(self.par, self.s, g, 0)

    def prepare(self, n_baby: int, n_groups: int):
        ck, plan, par = self.ckks, self.plan, self.par
        self.baby_ks = list(range(1, plan.b))[:n_baby]
        self.groups = [(pj % self.n_out, pj // self.n_out) for pj in range(self.n_out * plan.g)][-n_groups:]
        for k in self.baby_ks:
            self.key_for(k * plan.tau)
        for (_, j) in self.groups:
            self.key_for(j * plan.b * plan.tau)
        # encoded diagonals of the sampled groups (weights are cached: encoding is outside the step)
        for (p, j) in self.groups:
            for q in range(self.n_in):
                for k in range(plan.b):
                    if (p, q, j, k) not in self.encoded:
                        z = ck.plain_slots(self.W, plan, p, q, j, k, par.n)
                        self.encoded[(p, q, j, k)] = ck.to_residues(ck.encode_coeffs(z, par.N, par.scale),
                                                                    par.basis if plan.hoist == "double" else par.primes)
        # evaluation-domain inputs for the sampled inner sums (unrotated stand-ins keep this bounded); with double
        # hoisting they carry a residue modulo the special prime as well
        if plan.hoist == "double":
            ext = [self.np.concatenate([ct, ct[:, :1] % self.np.uint64(par.P)], axis=1) for ct in self.cts]
            self.Xh = [[ck.ntt(ext[q], par.basis * 2, par) for _ in range(plan.b)] for q in range(self.n_in)]
        else:
            self.Xh = [[ck.ntt(self.cts[q], par.primes * 2, par) for _ in range(plan.b)] for q in range(self.n_in)]

    def step(self) -> dict:
        """One sampled step; returns seconds per part and the unit counts they cover."""
        ck, plan, par = self.ckks, self.plan, self.par
        t = {"baby": 0.0, "inner": 0.0, "giant": 0.0, "rescale": 0.0}
        t0 = time.perf_counter()
        (ck.baby_rotations_ext if plan.hoist == "double" else ck.baby_rotations)(par, plan, self.cts[0], self.keys,
                                                                                  ks=self.baby_ks)
        t["baby"] = time.perf_counter() - t0
        n_giant = 0
        A = u = None
        for (p, j) in self.groups:
            t0 = time.perf_counter()
            A = ck.inner_sum(par, plan, self.Xh, self.encoded, p, j)
            t1 = time.perf_counter()
            t["inner"] += t1 - t0
            if j > 0:
                steps = j * plan.b * plan.tau
                if plan.moddown == "per_output":        # key switch without its own division by P
                    g = ck.galois_element(steps, par.N)
                    u = ck.key_switch_ext(par, A[1], g, self.keys[g])
                    for i, qi in enumerate(par.primes):
                        ck.automorphism(A[0, i], g, qi)
                else:
                    A = ck.rotate(par, A, steps, self.keys)
                t["giant"] += time.perf_counter() - t1
                n_giant += 1
        t0 = time.perf_counter()
        if u is not None:                               # the one division by P of an output, then its rescale
            ck.mod_down(u[0], par)
            ck.mod_down(u[1], par)
        ck.rescale(par, A)
        t["rescale"] = time.perf_counter() - t0
        t["n_baby"], t["n_inner"], t["n_giant"] = len(self.baby_ks), len(self.groups), max(1, n_giant)
        return t

    def scale_to_token(self, t: dict) -> float:
        """ms per decode token of the whole workload, scaling the sampled parts by unit counts:
        baby rotations per input ciphertext, inner sums per (block, giant step) group (their cost
        grows with the number of input chunks), giant rotations, one rescale per output block."""
        from paper_2606_17421_b200 import workloads as wl
        plan = self.plan
        per_baby = t["baby"] / t["n_baby"]
        per_inner = t["inner"] / t["n_inner"]
        per_giant = t["giant"] / t["n_giant"]
        total = 0.0
        spec = wl.PlanSpec(plan.D, plan.tau, plan.b, plan.g, plan.pack, plan.moddown, plan.hoist)
        # the calls the runner issues: projections that share an input stacked, each under its baby/giant split (an
        # inner sum has n_in * b terms: its sampled cost is scaled by both)
        for name, d_in, members in wl.fuse_shared_inputs(self.w.layers, plan.D):
            b, g = self.w.split_of(name, spec)
            n_in, n_out = wl.ceil_div(d_in, plan.D), plan.n_out(sum(m.d_out for m in members))
            total += n_in * (b - 1) * per_baby
            total += n_out * g * per_inner * (n_in / self.n_in) * (b / plan.b)
            total += n_out * (g - 1) * per_giant
            total += n_out * t["rescale"]
        return total * self.w.n_repeat * 1e3

    def size_sample(self, per_step_budget_s: float):
        """Pick how many baby rotations and groups one step covers so that it fits the budget."""
        self.prepare(1, 1)
        t = self.step()
        tb = max(t["baby"], 1e-3)
        tg = max(t["inner"] + t["giant"], 1e-3)
        n_baby = max(1, min(self.plan.b - 1, int(0.3 * per_step_budget_s / tb)))
        n_groups = max(1, min(self.n_out * self.plan.g, int(0.7 * per_step_budget_s / tg)))
        self.prepare(n_baby, n_groups)

    def describe(self) -> str:
        return (f"plan pack={self.plan.pack} moddown={self.plan.moddown} hoist={self.plan.hoist}; layer {self.L.name}: {len(self.baby_ks)} of {self.plan.b - 1} baby rotations of one input and "
                f"{len(self.groups)} of {self.n_out * self.plan.g} (block, giant-step) groups (inner sum, giant "
                f"rotation) plus one rescale per step, scaled by unit counts to every call of the workload (stacked projections, per-call splits)")


def cpu_baseline(workload: str, budget_s: float) -> dict:
    from oracle import ckks
    S = OracleSample(workload)
    cores = ckks.lib().orc_num_threads()
    S.size_sample(budget_s)
    t = S.step()
    secs = t["baby"] + t["inner"] + t["giant"] + t["rescale"]
    return {"value": round(S.scale_to_token(t), 2), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": S.describe() + f"; sampled work took {secs:.1f} s"}


def run_reference(args):
    """The reference arm of this build is the CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ckks
    S = OracleSample(args.workload)
    cores = ckks.lib().orc_num_threads()
    # size the per-step sample so that the whole run stays near two minutes
    S.size_sample(max(0.3, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        S.step()
    acc = None
    wall0 = time.perf_counter()
    for _ in range(args.steps):
        t = S.step()
        acc = t if acc is None else {k: (acc[k] + v if k in ("baby", "inner", "giant", "rescale") else v)
                                     for k, v in t.items()}
    wall = time.perf_counter() - wall0
    mean = {k: (v / args.steps if k in ("baby", "inner", "giant", "rescale") else v) for k, v in acc.items()}
    value = S.scale_to_token(mean)
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(wall / args.steps * 1e3, 2), "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": {"workload": args.workload},
            "cpu_baseline": {"value": round(value, 2), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": S.describe()},
            "e2e": {"value": round(value, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD,
                    help="workload[@option,...]: see parse_spec; default = the largest single-GPU configuration")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extra", default=DEFAULT_EXTRA,
                    help="comma-separated further workload specs timed after the main one (N=1 only); '' for none; "
                         "tiles = the tile-size study and the paper's own parameter set")
    args = ap.parse_args()
    if args.extra == "tiles":     # tile-size study and the paper's own parameter set
        args.extra = ("gemm1024_D1024,gemm1024_D512,gemm1024_D256,gemm1024_D128,gpt2_qkv_paper_params,"
                      "gpt2_qkv@fold")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
