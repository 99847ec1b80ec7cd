"""Drive the library over a workload with synthetic inputs (benchmarks and demos).

Holds no arithmetic of the method: it creates a context, fills rotation keys and ciphertexts with
seeded uniform residues (a fresh ciphertext or a switching key is indistinguishable from that, and
the kernels' work does not depend on the values), draws fp32 weights ~ N(0, 0.02^2), and calls the
C ABI.  Correctness is established elsewhere (tests compare with the CPU reference).
"""
from __future__ import annotations

import numpy as np
import torch

from . import bifrost as bf
from . import workloads as wl


def _uniform_residues(gen: torch.Generator, moduli, lead_shape, N: int, device) -> torch.Tensor:
    """int64 tensor [*lead_shape, len(moduli), N], slice m uniform in [0, moduli[m])."""
    out = torch.empty((*lead_shape, len(moduli), N), dtype=torch.int64, device=device)
    for m, q in enumerate(moduli):
        out[..., m, :] = torch.randint(0, int(q), (*lead_shape, N), generator=gen, device=device, dtype=torch.int64)
    return out


class WorkloadRunner:
    """One context per workload; per layer: weights (cached when the budget allows), input and
    output ciphertext buffers."""

    def __init__(self, name: str, seed: int = 0, device: str = "cuda:0", cache: bool = True,
                 cache_budget_bytes: int | None = None, stream: torch.cuda.Stream | None = None,
                 fuse_shared_inputs: bool = True, fold_in_ciphertext: bool = False, compact_cache: bool = False,
                 pack: str | None = None, moddown: str | None = None, hoist: str | None = None, coef_bits: int = 0,
                 lanes: int | None = None):
        self.w = wl.WORKLOADS[name]
        ps = wl.PARAM_SETS[self.w.params]
        self.N, self.primes, self.P, self.scale = ps["N"], list(ps["primes"]), ps["special"], ps["scale"]
        self.r = len(self.primes)
        self.plan = self.w.plan
        if pack or moddown or hoist:         # the workload's plan with another packing / key-switch variant
            self.plan = wl.PlanSpec(self.plan.D, self.plan.tau, self.plan.b, self.plan.g,
                                    pack or self.plan.pack, moddown or self.plan.moddown, hoist or self.plan.hoist)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        # a stream of our own: the legacy default stream cannot be captured, which would keep the
        # library from replaying its launch sequences as CUDA graphs
        self.stream = stream or torch.cuda.Stream(device=self.device)
        torch.cuda.set_stream(self.stream)
        self.gen = torch.Generator(device=self.device)
        self.gen.manual_seed(seed)
        self.ctx = bf.bf_ctx_create(self.N, self.primes + [self.P], self.r, self.scale,
                                    bf.bf_plan(self.plan.D, self.plan.tau, self.plan.b, self.plan.g,
                                               (bf.BF_PLAN_COMPLEX_PACK if self.plan.pack == "complex" else 0) |
                                               (bf.BF_PLAN_MODDOWN_PER_OUTPUT if self.plan.moddown == "per_output" else 0) |
                                               (bf.BF_PLAN_DOUBLE_HOIST if self.plan.hoist == "double" else 0)),
                                    self.stream.cuda_stream)
        if compact_cache:           # narrower resident words per prime: 68 % of the cache for the 50 + 6 x 40-bit chain
            bf.bf_set_compact_cache(self.ctx, True)
        self.compact_cache = compact_cache
        if lanes:                   # concurrent key-switch chains (the library's default otherwise)
            bf.bf_set_lanes(self.ctx, lanes)
        if coef_bits:               # weights resident as rounded 64- or 32-bit coefficients, transformed on every call
            bf.bf_set_coefficient_cache(self.ctx, coef_bits)
        self.coef_bits = coef_bits
        # resident bytes per encoded coefficient over all primes (8 each, or 4 / 5 / 8 by prime size when compact)
        self.word_bytes = sum((4 if q < 2 ** 32 else 5 if q < 2 ** 40 else 8) if compact_cache else 8 for q in self.primes)
        if self.plan.hoist == "double":     # the residue modulo the special prime is kept too, always in 8 bytes
            self.word_bytes += 8
        budget = cache_budget_bytes if cache_budget_bytes is not None else self.w.cache_budget_bytes
        if budget:
            bf.bf_set_cache_budget(self.ctx, int(budget))
        # calls: projections that read the same activation stacked into one (q/k/v, gate/up), each with its baby/giant split
        D = self.plan.D
        if fuse_shared_inputs:
            fused = wl.fuse_shared_inputs(self.w.layers, D)
            units = [wl.Layer(nm, d_in, sum(m.d_out for m in members)) for nm, d_in, members in fused]
            members_of = {nm: members for nm, _, members in fused}
        else:
            units = list(self.w.layers)
            members_of = {L.name: [L] for L in units}
        self.splits = {L.name: self.w.split_of(L.name, self.plan) for L in units}
        # rotation keys for every split in use: uniform residues over the extended basis
        steps = []
        for b, g in sorted(set(self.splits.values()) | {(self.plan.b, self.plan.g)}):
            steps += [k * self.plan.tau for k in range(1, b)] + [j * b * self.plan.tau for j in range(1, g)]
        self.fold_in_ciphertext = fold_in_ciphertext
        if fold_in_ciphertext:      # the variant that sums the tau partial results on the device
            steps += [1 << i for i in range(self.plan.tau.bit_length() - 1)]
        n = self.N // 2
        self.rot_steps = sorted({s % n for s in steps if s % n})
        basis = self.primes + [self.P]
        if self.rot_steps:
            keys = _uniform_residues(self.gen, basis, (len(self.rot_steps), self.r, 2), self.N, self.device)
            bf.bf_load_eval_keys(self.ctx, self.rot_steps, len(self.rot_steps), keys)
            del keys
        self.key_bytes = len(self.rot_steps) * self.r * 2 * (self.r + 1) * self.N * 8
        # layers
        self.layers = []
        for rep in range(self.w.n_repeat):
            for L in units:
                n_in, n_out = wl.ceil_div(L.d_in, D), wl.ceil_div(L.d_out, self.plan.rows_per_ct)
                W = torch.from_numpy(np.concatenate(
                    [wl.gen_weights(seed, f"{m.name}.{rep}", m.d_out, m.d_in) for m in members_of[L.name]], axis=0)
                ).to(self.device)
                handle = None
                b, g = self.splits[L.name]
                if cache:
                    try:
                        handle = bf.bf_encode_weights_split(self.ctx, W, L.d_out, L.d_in, b, g)
                    except bf.BifrostError as e:
                        if e.code != bf.BF_ERR_OOM:
                            raise
                if handle is None:      # the on-the-fly path runs under the plan's own split
                    b, g = self.plan.b, self.plan.g
                ct_in = _uniform_residues(self.gen, self.primes, (n_in, 2), self.N, self.device)
                ct_out = torch.empty((n_out, 2, self.r, self.N), dtype=torch.int64, device=self.device)
                ct_low = torch.empty((n_out, 2, self.r - 1, self.N), dtype=torch.int64, device=self.device)
                self.layers.append(dict(layer=L, rep=rep, n_in=n_in, n_out=n_out, b=b, g=g, W=W, handle=handle,
                                        ct_in=ct_in, ct_out=ct_out, ct_low=ct_low,
                                        pt_bytes=n_in * n_out * (D // self.plan.tau) * self.N * self.word_bytes,
                                        resident_bytes=n_in * n_out * (D // self.plan.tau) * self.N *
                                        (coef_bits // 8 if coef_bits else self.word_bytes) if handle else 0))
        torch.cuda.synchronize()

    # ------------------------------------------------------------------ one decode token
    def step(self):
        """All linear layers of the workload once: the product and its rescale per layer (device buffers), as the one
        call that does both unless the in-ciphertext fold sits between them."""
        for e in self.layers:
            L = e["layer"]
            if not self.fold_in_ciphertext:
                bf.bf_linear_rescaled(self.ctx, e["ct_in"], e["n_in"], e["handle"], None if e["handle"] else e["W"],
                                      L.d_out, L.d_in, e["ct_low"], e["n_out"])
                continue
            bf.bf_linear(self.ctx, e["ct_in"], e["n_in"], e["handle"], None if e["handle"] else e["W"],
                         L.d_out, L.d_in, e["ct_out"], e["n_out"])
            bf.bf_fold(self.ctx, e["ct_out"], e["n_out"])
            bf.bf_rescale(self.ctx, e["ct_out"], e["ct_low"], e["n_out"], self.r)

    def make_host_buffers(self):
        for e in self.layers:
            e["h_in"] = e["ct_in"].cpu().pin_memory()
            e["h_out"] = torch.empty((e["n_out"], 2, self.r - 1, self.N), dtype=torch.int64).pin_memory()

    def step_host(self):
        """The same through the host-buffer entry point: ciphertexts travel host -> device -> host."""
        for e in self.layers:
            L = e["layer"]
            bf.bf_linear_host(self.ctx, e["h_in"], e["n_in"], e["handle"], None if e["handle"] else e["W"],
                              L.d_out, L.d_in, e["h_out"], e["n_out"])

    def host_bytes_per_step(self):
        h2d = sum(e["n_in"] * 2 * self.r * self.N * 8 for e in self.layers)
        d2h = sum(e["n_out"] * 2 * (self.r - 1) * self.N * 8 for e in self.layers)
        return h2d, d2h

    def cached_pt_bytes(self):
        return sum(e["pt_bytes"] for e in self.layers if e["handle"])

    def resident_bytes(self):
        """Bytes the cached weights occupy (differs from the streamed bytes when they are kept as coefficients)."""
        return sum(e["resident_bytes"] for e in self.layers)

    def total_pt_bytes(self):
        return sum(e["pt_bytes"] for e in self.layers)

    def n_fallback_layers(self):
        return sum(1 for e in self.layers if not e["handle"])

    def transforms_weights_per_call(self, e) -> bool:
        """The call of layer entry e transforms its weights (encoded on the fly, or kept as coefficients)."""
        return not e["handle"] or bool(self.coef_bits)

    def close(self):
        bf.bf_ctx_destroy(self.ctx)
        self.layers = []
