"""Workload definitions and seeded synthetic inputs.

This module holds NONE of the method's arithmetic: only shapes, CKKS parameter literals and
random-number recipes.  It is the one module both the CPU reference used by the tests and the CUDA
library's callers draw inputs from.

The synthetic layers stand in for the trained GPT-2 / Qwen3 / LLaMA-3 checkpoints the paper's
evaluation (Sec. 5.1) runs on: only the layer shapes are kept; weights are fp32 N(0, 0.02^2),
activations fp64 N(0, 1), everything derived from one base seed with a distinct stream per object.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field

import numpy as np

# ----------------------------------------------------------------------------- CKKS parameter sets
# Largest primes = 1 (mod 2N) below 2^50 (base prime), below 2^40 (descending) and below 2^60
# (special prime for key switching).
Q40_N15 = [1099510054913, 1099507695617, 1099506515969, 1099504549889, 1099503894529, 1099503370241]

PARAM_SETS = {
    "n12": dict(N=1 << 12, primes=[1125899906826241, 1099511480321, 1099511390209],
                special=1152921504606830593, scale=2.0 ** 40),
    "n15": dict(N=1 << 15, primes=[1125899904679937] + Q40_N15,
                special=1152921504606584833, scale=2.0 ** 40),
    "n16": dict(N=1 << 16, primes=[1125899903827969] + Q40_N15 + [1099502714881, 1099500617729],
                special=1152921504606584833, scale=2.0 ** 40),
    # The prototype's own parameter set (Sec. 4.2): N = 8192, primes of [60, 30, 30, 30] bits,
    # scale 2^30, one 60-bit special prime.
    "paper_n13": dict(N=1 << 13, primes=[1152921504606830593, 1073692673, 1073643521, 1073479681],
                      special=1152921504606748673, scale=2.0 ** 30),
}


@dataclass(frozen=True)
class PlanSpec:
    """Tile side D, replica split tau, baby steps b, giant steps g (b*g = D/tau)."""
    D: int
    tau: int
    b: int
    g: int
    pack: str = "real"                  # "complex": two output row blocks per plaintext (real and imaginary parts)
    moddown: str = "per_rotation"       # "per_output": one division by the special prime per output ciphertext
    hoist: str = "single"               # "double": baby-step rotations stay in the extended basis, one division per inner sum

    @property
    def rows_per_ct(self) -> int:
        return self.D * (2 if self.pack == "complex" else 1)


@dataclass(frozen=True)
class Layer:
    name: str
    d_in: int
    d_out: int
    input: str = ""             # projections of one transformer layer with the same non-empty tag read the same
                                # activation: a caller may stack their weight matrices row-wise into one call
                                # (output row blocks are independent, so every residue is unchanged)


@dataclass(frozen=True)
class Workload:
    name: str
    params: str                 # key of PARAM_SETS
    plan: PlanSpec
    layers: tuple               # the distinct projections of one transformer layer
    n_repeat: int = 1           # number of transformer layers in a decode step
    cache_budget_bytes: int | None = None
    # baby/giant splits (b, g) of single calls (by the name of the call, stacked projections joined with "+") that differ
    # from the plan's: measured per call shape on B200 under double hoisting with one division per output, and used
    # under that plan variant only.  Many input ciphertexts favour fewer baby steps, many outputs fewer giant steps.
    splits: dict = field(default_factory=dict)

    def split_of(self, call: str, plan: PlanSpec):
        if plan.hoist == "double" and plan.moddown == "per_output":
            return self.splits.get(call, (plan.b, plan.g))
        return (plan.b, plan.g)


GPT2_LAYER = (Layer("qkv", 768, 2304), Layer("out_proj", 768, 768),
              Layer("ffn_up", 768, 3072), Layer("ffn_down", 3072, 768))
QWEN3_LAYER = (Layer("q", 1024, 2048, "attn"), Layer("k", 1024, 1024, "attn"), Layer("v", 1024, 1024, "attn"),
               Layer("o", 2048, 1024), Layer("gate", 1024, 3072, "ffn"), Layer("up", 1024, 3072, "ffn"),
               Layer("down", 3072, 1024))
LLAMA3_8B_LAYER = (Layer("q", 4096, 4096, "attn"), Layer("k", 4096, 1024, "attn"), Layer("v", 4096, 1024, "attn"),
                   Layer("o", 4096, 4096), Layer("gate", 4096, 14336, "ffn"), Layer("up", 4096, 14336, "ffn"),
                   Layer("down", 14336, 4096))


def fuse_shared_inputs(layers, D: int):
    """Group consecutive projections that read the same activation: [(fused name, d_in, [member layers])].
    Members must have d_out a multiple of the tile side D so that their row blocks stay aligned."""
    groups = []
    for L in layers:
        if groups and L.input and groups[-1][2][-1].input == L.input and groups[-1][1] == L.d_in \
                and all(m.d_out % D == 0 for m in groups[-1][2]):
            groups[-1][2].append(L)
            groups[-1][0] += "+" + L.name
        else:
            groups.append([L.name, L.d_in, [L]])
    return [(name, d_in, members) for name, d_in, members in groups]

WORKLOADS = {
    "tiny": Workload("tiny", "n12", PlanSpec(64, 1, 8, 8), (Layer("w", 64, 64),)),
    # M = 64 diagonals per tile split as 16 baby x 4 giant steps: measured fastest on B200 (fewer full
    # key switches than 8 x 8 at the price of four more rotation keys)
    "gpt2_qkv": Workload("gpt2_qkv", "n15", PlanSpec(1024, 16, 16, 4), (GPT2_LAYER[0],)),
    # (per call, ms on B200 for 16x4 / 32x2 / 8x8: ffn_down 0.507 / 0.872 / 0.490; the other three are fastest at 16x4)
    "gpt2_step": Workload("gpt2_step", "n15", PlanSpec(1024, 16, 16, 4), GPT2_LAYER, n_repeat=12,
                          splits={"ffn_down": (8, 8)}),
    # (16x4 / 32x2 / 8x8: q+k+v 0.380 / 0.395 / 0.534, o 0.384 / 0.535 / 0.401, gate+up 0.483 / 0.454 / 0.729,
    # down 0.507 / 0.872 / 0.490)
    "qwen3_step": Workload("qwen3_step", "n15", PlanSpec(1024, 16, 16, 4), QWEN3_LAYER, n_repeat=28,
                           cache_budget_bytes=60 * 10 ** 9, splits={"gate+up": (32, 2), "down": (8, 8)}),
    # (8x4 / 16x2 / 4x8: q+k+v 1.79 / 1.79 / 2.49, o 1.43 / 1.56 / 1.84, gate+up 5.88 / 4.25 / 9.86,
    # down 3.78 / 6.29 / 3.44)
    "llama3_layer": Workload("llama3_layer", "n16", PlanSpec(1024, 32, 8, 4), LLAMA3_8B_LAYER,
                             splits={"gate+up": (16, 2), "down": (4, 8)}),
}
# Tile-size study (the paper's Sec. 5.3 experiment on a 1024 x 1024 product): smaller tiles need fewer or no
# rotations but send more ciphertexts across the TEE boundary (1024/D in, 1024/D out).
for _D, _tau, _b, _g in ((1024, 16, 16, 4), (512, 32, 4, 4), (256, 64, 2, 2), (128, 128, 1, 1)):
    WORKLOADS[f"gemm1024_D{_D}"] = Workload(f"gemm1024_D{_D}", "n15", PlanSpec(_D, _tau, _b, _g),
                                            (Layer("w", 1024, 1024),))
# The GPT-2 QKV projection under the prototype's own CKKS parameters (Sec. 4.2): N = 8192, 4096 slots.
WORKLOADS["gpt2_qkv_paper_params"] = Workload("gpt2_qkv_paper_params", "paper_n13", PlanSpec(1024, 4, 16, 16),
                                              (GPT2_LAYER[0],))
# One transformer layer of the GPT-2 step (1.2 GB of encoded weights): small enough for profiler captures that need
# several passes, with the call shapes of the whole step (one and three input ciphertexts, one and three output blocks).
WORKLOADS["gpt2_layer"] = Workload("gpt2_layer", "n15", PlanSpec(1024, 16, 16, 4), GPT2_LAYER,
                                   splits={"ffn_down": (8, 8)})
CONFIG_ORDER = ["tiny", "gpt2_qkv", "gpt2_step", "qwen3_step", "llama3_layer"]


# ----------------------------------------------------------------------------- seeded generators

def _stream(seed: int, *tag) -> np.random.Generator:
    words = [seed & 0xFFFFFFFF]
    for t in tag:
        words.append(zlib.crc32(str(t).encode()) if not isinstance(t, int) else t & 0xFFFFFFFF)
    return np.random.Generator(np.random.PCG64(words))


def gen_weights(seed: int, tag, d_out: int, d_in: int) -> np.ndarray:
    """fp32 W[d_out][d_in] ~ N(0, 0.02^2)."""
    return (_stream(seed, "W", tag).standard_normal((d_out, d_in)) * 0.02).astype(np.float32)


def gen_activation(seed: int, tag, d_in: int) -> np.ndarray:
    """fp64 x[d_in] ~ N(0, 1)."""
    return _stream(seed, "x", tag).standard_normal(d_in)


def gen_uniform_residues(seed: int, tag, moduli, shape_tail) -> np.ndarray:
    """uint64 [len(moduli), *shape_tail], row i uniform in [0, moduli[i]).  A fresh ciphertext and a
    switching key are computationally indistinguishable from this, so it serves as a stand-in
    when only throughput is measured."""
    rng = _stream(seed, "u", tag)
    return np.stack([rng.integers(0, int(q), size=shape_tail, dtype=np.uint64) for q in moduli])


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)
