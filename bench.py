#!/usr/bin/env python
"""Benchmark of the encrypted linear layer: ms per decode token on one B200 (or N independent
replicas, one process per GPU), with the roofline of the dominant kernels and the CPU oracle
timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload gpt2_qkv] [--impl reference]

A step = one decode token's worth of the workload: bf_linear + bf_rescale for every linear layer
of the workload, cached encoded weights streamed from HBM (352 MB per step for gpt2_qkv, larger
than L2, so consecutive steps cannot be served from cache).  Inputs are seeded and synthetic.
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

# DRAM bytes (read + write) per launch of the named kernel from an ncu capture of this workload;
# see profiles/ for the capture each figure comes from.  None = not captured yet.
NCU_TRAFFIC_BYTES = {
    # from the ncu capture summarised under profiles/: dram__bytes_read.sum + dram__bytes_write.sum per launch
    "gpt2_qkv": {"mac": 423.7e6,                       # 411.1 MB read + 12.6 MB written
                 "key_inner_product": 373.1e6,         # 746 MB per step (two lanes' launches), over the two launches of
                                                       #   the serialised timing pass
                 "ntt_fwd_strided": 23.8e6,            # mean of the eight captured forward launches (both passes)
                 "ntt_inv_contig": 11.0e6},            # mean of the eight captured inverse launches (both passes)
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


def butterflies_per_step(runner) -> dict:
    """Transforms one step launches, by direction and by arithmetic path.  Moduli below 2^41 run in
    fp64 with 8 fp64 operations per butterfly (signed lazy values), moduli from 2^41 up to 2^50 in fp64
    with a conditional subtraction and offsets (12 operations), the 60-bit special prime in integers
    (at least 10 32-bit multiply-adds per butterfly); both pipes issue 64 lanes per clock per SM."""
    import math
    r, N = runner.r, runner.N
    b, g = runner.plan.b, runner.plan.g
    per = (N // 2) * int(math.log2(N))
    moduli = list(runner.primes) + [runner.P]
    cost = [8 if q < (1 << 41) else 12 if q < (1 << 50) else 10 for q in moduli]
    fp = [q < (1 << 50) for q in moduli]
    fwd = [0] * (r + 1)
    inv = [0] * (r + 1)
    for e in runner.layers:
        n_in, n_out = e["n_in"], e["n_out"]
        n_giant = (g - 1) * n_out
        sets = (n_in if b > 1 else 0) + n_giant            # ModUp digit sets
        rots = n_in * (b - 1) + n_giant                    # key switches
        for i in range(r):
            fwd[i] += 2 * n_in + sets * (r - 1) + 2 * rots # inputs; digits of the other primes; lifted P-residues
            inv[i] += n_giant + 2 * n_out                  # c1 of the giant-step inputs; outputs
        fwd[r] += sets * r
        inv[r] += 2 * rots                                 # P-residues of the inner products
    def summary(cnt):
        polys = sum(cnt)
        ops = sum(c * k for c, k in zip(cnt, cost))
        return {"polys": polys, "fp64_polys": sum(c for c, f in zip(cnt, fp) if f), "ops_per_butterfly": ops / max(1, polys)}
    return {"fwd": summary(fwd), "inv": summary(inv), "per_poly": per}


def time_extra_workload(name: str, steps: int, cache_budget_bytes=None, fold_in_ciphertext=False,
                        compact_cache=False) -> dict:
    """ms per decode token of another workload (device-resident inputs), with the weight stream's rate."""
    import torch
    from paper_2606_17421_b200 import bifrost as bf
    from paper_2606_17421_b200.runner import WorkloadRunner
    R = WorkloadRunner(name, cache_budget_bytes=cache_budget_bytes, fold_in_ciphertext=fold_in_ciphertext,
                       compact_cache=compact_cache)
    for _ in range(3):
        R.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        R.step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    bf.bf_get_kernel_stats(R.ctx)
    bf.bf_set_kernel_timing(R.ctx, True)
    bf.bf_set_lanes(R.ctx, 1)              # one chain: every kernel runs alone, so its event pair times it alone
    for _ in range(steps):
        R.step()
    st = bf.bf_get_kernel_stats(R.ctx)
    bf.bf_set_lanes(R.ctx, DEFAULT_LANES)
    mac_n, mac_ms = st["mac"]
    enc_ms = (st["encode_fft_a"][1] + st["encode_fft_b"][1]) / steps
    h2d, d2h = R.host_bytes_per_step()
    out = {"ms_per_token": round(ms, 4), "layers": len(R.layers),
           "ciphertexts_in": sum(e["n_in"] for e in R.layers), "ciphertexts_out": sum(e["n_out"] for e in R.layers),
           "boundary_bytes": h2d + d2h, "rotation_keys": len(R.rot_steps), "fallback_layers": R.n_fallback_layers(),
           "plan": {"D": R.plan.D, "tau": R.plan.tau, "b": R.plan.b, "g": R.plan.g},
           "encoded_weight_bytes_cached": R.cached_pt_bytes(), "encoded_weight_bytes_total": R.total_pt_bytes(),
           "mac_gbs": round(R.total_pt_bytes() * steps / (mac_ms * 1e-3) / 1e9, 1) if mac_ms else None,
           "kernel_ms_per_token": {k: round(v[1] / steps, 3) for k, v in st.items() if v[0]},
           "encode_fft_ms_per_token": round(enc_ms, 3)}
    R.close()
    torch.cuda.empty_cache()
    return out


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
    from paper_2606_17421_b200.runner import WorkloadRunner
    from paper_2606_17421_b200.replicas import job_ms_per_token, max_over_ranks

    bf.load()   # fails loudly when the CUDA library is missing
    # every rank decodes its own token stream (independent problems: no data-path collective)
    R = WorkloadRunner(args.workload, seed=rank, device=f"cuda:{local}")
    stream = R.stream                       # the runner's own stream, made torch's current stream

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        t1 = time.time()
        ms = max_over_ranks(e0.elapsed_time(e1), device="cuda")
        return ms, t0, t1

    for _ in range(max(args.warmup, 3)):
        R.step()
    barrier()
    bf.bf_get_kernel_stats(R.ctx)   # reset launch counters

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    ms_total, t0, t1 = timed(R.step, args.steps)
    stats = bf.bf_get_kernel_stats(R.ctx)
    gpu_launches = sum(v[0] for v in stats.values())
    ms_per_step = ms_total / args.steps

    # per-kernel durations: the same K steps again with an event pair around every launch, and with the
    # key-switch chains serialised (one lane) so that no other kernel of the step runs beside the timed one
    bf.bf_set_kernel_timing(R.ctx, True)
    bf.bf_set_lanes(R.ctx, 1)
    timed(R.step, args.steps)
    kstats = bf.bf_get_kernel_stats(R.ctx)
    bf.bf_set_kernel_timing(R.ctx, False)
    bf.bf_set_lanes(R.ctx, DEFAULT_LANES)

    # end to end through the host-buffer entry point (pinned host ciphertexts in and out)
    R.make_host_buffers()
    for _ in range(3):
        R.step_host()
    e2e_steps = max(3, min(args.steps, 50))
    e2e_total, _, _ = timed(R.step_host, e2e_steps)
    e2e_ms = e2e_total / e2e_steps
    sampler.stop()
    clocks = sampler.summary(t0, t1)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    hbm_peak, peak_kind = read_peaks()
    imad_rate = bf.bf_measure_imad_rate(R.ctx)
    bfly = butterflies_per_step(R)
    K = args.steps
    traffic = NCU_TRAFFIC_BYTES.get(args.workload, {})

    def avg_ms(cat):
        n, ms = kstats[cat]
        return (ms / n) if n else None, n / K

    rooflines = {}
    # weight-streaming multiply-accumulate: algorithmic bytes = every encoded word once
    mac_ms, mac_n = avg_ms("mac")
    if mac_ms:
        mac_bytes = R.cached_pt_bytes() / max(1.0, mac_n)
        ach = mac_bytes / (mac_ms * 1e-3) / 1e9
        rooflines["mac"] = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s",
                            "frac": round(ach / hbm_peak, 4), "of": peak_kind, "traffic": traffic.get("mac"),
                            "launches_per_step": mac_n, "avg_ms": round(mac_ms, 5),
                            "frac_of_nominal_8000": round(ach / 8000.0, 4)}
    # key-switch inner product: algorithmic bytes = the key stream of each rotation once
    ki_ms, ki_n = avg_ms("key_inner_product")
    if ki_ms:
        n_rot = sum(e["n_in"] * (R.plan.b - 1) + e["n_out"] * (R.plan.g - 1) for e in R.layers)
        key_bytes = n_rot * R.r * 2 * (R.r + 1) * R.N * 8 / max(1.0, ki_n)
        ach = key_bytes / (ki_ms * 1e-3) / 1e9
        rooflines["key_inner_product"] = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s",
                                          "frac": round(ach / hbm_peak, 4), "of": peak_kind,
                                          "traffic": traffic.get("key_inner_product"),
                                          "launches_per_step": ki_n, "avg_ms": round(ki_ms, 5),
                                          "note": "bytes = one key per rotation; rotations sharing a key hit L2"}
    # transforms: bound by the arithmetic pipes (fp64 for the ciphertext primes, integer multiply-add for the special prime)
    sm_mhz = clocks.get("sm_mhz") or 1965.0
    lanes_per_s = 148 * 64 * sm_mhz * 1e6                  # either pipe: 148 SMs x 64 lanes x clock
    for cats, key, label in ((("ntt_fwd_strided", "ntt_fwd_contig"), "fwd", "ntt_forward"),
                             (("ntt_inv_contig", "ntt_inv_strided"), "inv", "ntt_inverse")):
        ms_step = sum(kstats[c][1] for c in cats) / K
        if ms_step > 0:
            info = bfly[key]
            rate = info["polys"] * bfly["per_poly"] / (ms_step * 1e-3)
            peak = lanes_per_s / info["ops_per_butterfly"]
            rooflines[label] = {"bound": "alu", "achieved": round(rate / 1e9, 1), "peak": round(peak / 1e9, 1),
                                "unit": "G butterflies/s", "frac": round(rate / peak, 4),
                                "of": (f"derived: 148 SMs x 64 lanes x {sm_mhz:.0f} MHz / {info['ops_per_butterfly']:.2f} "
                                       "pipe operations per butterfly (8 fp64 ops below 2^41, 12 up to 2^50, 10 multiply-adds on "
                                       f"the integer path); bf_measure_imad_rate measured {imad_rate / 1e12:.2f} T multiply-adds/s"),
                                "traffic": traffic.get(cats[0]), "ms_per_step": round(ms_step, 5),
                                "polys_per_step": info["polys"], "fp64_polys_per_step": info["fp64_polys"]}
    total_k_ms = sum(v[1] for v in kstats.values())
    shares = {k: round(v[1] / total_k_ms, 4) for k, v in kstats.items() if v[0]}
    dominant = max(shares, key=shares.get)
    dom_key = {"ntt_fwd_strided": "ntt_forward", "ntt_fwd_contig": "ntt_forward", "ntt_inv_contig": "ntt_inverse",
               "ntt_inv_strided": "ntt_inverse"}.get(dominant, dominant)
    roofline = dict(rooflines.get(dom_key, rooflines.get("mac", {})))
    roofline["kernel"] = dom_key

    h2d, d2h = R.host_bytes_per_step()
    line = {
        "metric": METRIC, "value": round(job_ms_per_token(ms_per_step, world), 5), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5),
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": args.workload, "ring_N": R.N, "ct_primes": R.r,
                   "plan": {"D": R.plan.D, "tau": R.plan.tau, "b": R.plan.b, "g": R.plan.g},
                   "layers": len(R.layers), "encoded_weight_bytes_per_step": R.cached_pt_bytes(),
                   "fallback_layers": R.n_fallback_layers(),
                   "l2": "inputs larger than L2: the encoded weights streamed each step exceed 126 MB",
                   "multi_gpu": "replicas: every rank decodes its own token, no data-path collective"},
        "tokens_per_s": round(world * 1e3 / ms_per_step, 3),
        "clocks": clocks,
        "e2e": {"value": round(job_ms_per_token(e2e_ms, world), 5), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": gpu_launches,
        "roofline": roofline,
        "rooflines": rooflines,
        "kernel_time_share": shares,
        "kernel_timing": "event pair around every launch with the key-switch chains serialised (1 lane); "
                         f"value and e2e are timed with {DEFAULT_LANES} concurrent chains and no per-launch events",
        "imad_rate_per_sm_clk": round(imad_rate / 148 / ((clocks.get("sm_mhz") or 1965.0) * 1e6), 2),
    }
    R.close()
    torch.cuda.empty_cache()
    if world == 1 and args.extra:
        extras = {}
        for name in args.extra.split(","):
            if name == "qwen3_step":
                # 60 GB keeps every layer resident; 40.5 GB = 23/28 of the encoded size reproduces the
                # partially cached regime (Sec. 6.1, table "FHE decode cost breakdown"): the overflow layers are encoded on every call
                full = time_extra_workload(name, 5, cache_budget_bytes=60 * 10 ** 9)
                part = time_extra_workload(name, 3, cache_budget_bytes=int(40.5 * 10 ** 9))
                part["fallback_share_of_step"] = round(1.0 - full["ms_per_token"] / part["ms_per_token"], 4)
                extras[name + "@60GB"] = full
                extras[name + "@40.5GB"] = part
                # the same budget with the compact cache format: every layer fits, nothing falls back
                extras[name + "@40.5GB_compact_cache"] = time_extra_workload(name, 5, cache_budget_bytes=int(40.5 * 10 ** 9),
                                                                             compact_cache=True)
            elif name == "llama3_layer":
                extras[name + "@cached"] = time_extra_workload(name, 5)
                extras[name + "@on_the_fly"] = time_extra_workload(name, 3, cache_budget_bytes=1)
            elif name == "gpt2_qkv@on_the_fly":
                # the headline call with its weights encoded inside the call (fallback path)
                extras[name] = time_extra_workload("gpt2_qkv", 50, cache_budget_bytes=1)
            elif name == "gpt2_qkv@fold_in_ciphertext":
                # the variant that sums the tau partial results on the device (log2 tau more key switches)
                extras[name] = time_extra_workload("gpt2_qkv", 50, fold_in_ciphertext=True)
            else:
                extras[name] = time_extra_workload(name, 10)
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

    def __init__(self, workload: str):
        import numpy as np
        from oracle import ckks
        from paper_2606_17421_b200 import workloads as wl
        self.np, self.ckks = np, ckks
        w = wl.WORKLOADS[workload]
        ps = wl.PARAM_SETS[w.params]
        self.w = w
        self.par = ckks.Params(ps["N"], list(ps["primes"]), ps["special"], ps["scale"])
        self.plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g)
        self.L = w.layers[0]
        self.W = wl.gen_weights(0, self.L.name, self.L.d_out, self.L.d_in)
        x = wl.gen_activation(0, self.L.name, self.L.d_in)
        self.s = ckks.keygen(self.par, 0)
        self.cts = ckks.encrypt_vector(self.par, self.plan, self.s, x, 0)
        self.keys = {}
        self.n_in = len(self.cts)
        self.n_out = -(-self.L.d_out // self.plan.D)
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
                        z = ck.bsgs_plain_slots(self.W, plan, p, q, j, k, par.n)
                        self.encoded[(p, q, j, k)] = ck.to_residues(ck.encode_coeffs(z, par.N, par.scale), par.primes)
        # evaluation-domain inputs for the sampled inner sums (unrotated stand-ins keep this bounded)
        self.Xh = [[ck.ntt(self.cts[q], par.primes * 2, par) for _ in range(plan.b)] for q in range(self.n_in)]

    def step(self) -> dict:
        """One sampled step; returns seconds per part and the unit counts they cover."""
        ck, plan, par = self.ckks, self.plan, self.par
        t = {"baby": 0.0, "inner": 0.0, "giant": 0.0, "rescale": 0.0}
        t0 = time.perf_counter()
        ck.baby_rotations(par, plan, self.cts[0], self.keys, ks=self.baby_ks)
        t["baby"] = time.perf_counter() - t0
        n_giant = 0
        A = None
        for (p, j) in self.groups:
            t0 = time.perf_counter()
            A = ck.inner_sum(par, plan, self.Xh, self.encoded, p, j)
            t1 = time.perf_counter()
            t["inner"] += t1 - t0
            if j > 0:
                A = ck.rotate(par, A, j * plan.b * plan.tau, self.keys)
                t["giant"] += time.perf_counter() - t1
                n_giant += 1
        t0 = time.perf_counter()
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
        for L in self.w.layers:
            n_in, n_out = wl.ceil_div(L.d_in, plan.D), wl.ceil_div(L.d_out, plan.D)
            total += n_in * (plan.b - 1) * per_baby
            total += n_out * plan.g * per_inner * (n_in / self.n_in)
            total += n_out * (plan.g - 1) * per_giant
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
        return (f"layer {self.L.name}: {len(self.baby_ks)} of {self.plan.b - 1} baby rotations of one input and "
                f"{len(self.groups)} of {self.n_out * self.plan.g} (block, giant-step) groups (inner sum, giant "
                f"rotation) plus one rescale per step, scaled by unit counts to every layer of the workload")


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
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="gpt2_qkv")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extra", default="gpt2_step",
                    help="comma-separated further workloads timed after the main one (N=1 only); '' for none; "
                         "all = gpt2_qkv@on_the_fly,gpt2_step,qwen3_step,llama3_layer")
    args = ap.parse_args()
    if args.extra == "all":
        args.extra = "gpt2_qkv@on_the_fly,gpt2_step,qwen3_step,llama3_layer"
    elif args.extra == "tiles":     # tile-size study and the paper's own parameter set
        args.extra = ("gemm1024_D1024,gemm1024_D512,gemm1024_D256,gemm1024_D128,gpt2_qkv_paper_params,"
                      "gpt2_qkv@fold_in_ciphertext")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
