"""Shared set-up for the GPU parity tests: oracle-side objects and the matching library context."""
import numpy as np

from oracle import ckks
from paper_2606_17421_b200 import workloads as wl


def oracle_params(param_key: str) -> ckks.Params:
    ps = wl.PARAM_SETS[param_key]
    return ckks.Params(ps["N"], list(ps["primes"]), ps["special"], ps["scale"])


def custom_params(N: int, n_small: int, scale=2.0 ** 40) -> ckks.Params:
    primes, P = ckks.prime_chain(N, n_small)
    return ckks.Params(N, primes, P, scale)


class GpuSide:
    """A library context plus torch helpers.  Imported lazily so CPU-only runs never touch CUDA."""

    def __init__(self, par: ckks.Params, plan: ckks.Plan):
        import torch
        from paper_2606_17421_b200 import bifrost as bf
        self.torch, self.bf = torch, bf
        self.par, self.plan = par, plan
        self.dev = torch.device("cuda:0")
        # work on a stream of our own: the legacy default stream cannot be captured, and bf_linear
        # replays captured launch sequences
        self.stream = torch.cuda.Stream(device=self.dev)
        torch.cuda.set_stream(self.stream)
        flags = (bf.BF_PLAN_COMPLEX_PACK if plan.pack == "complex" else 0) | \
                (bf.BF_PLAN_MODDOWN_PER_OUTPUT if plan.moddown == "per_output" else 0) | \
                (bf.BF_PLAN_DOUBLE_HOIST if plan.hoist == "double" else 0)
        p = bf.bf_plan(plan.D, plan.tau, plan.b, plan.g, flags)
        self.ctx = bf.bf_ctx_create(par.N, par.basis, par.r, par.scale, p,
                                    torch.cuda.current_stream().cuda_stream)

    def close(self):
        self.bf.bf_ctx_destroy(self.ctx)

    def to_dev(self, a: np.ndarray):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint64:
            return self.torch.from_numpy(a.view(np.int64)).to(self.dev)
        return self.torch.from_numpy(a).to(self.dev)

    def to_host_u64(self, t) -> np.ndarray:
        self.torch.cuda.synchronize()
        return t.cpu().numpy().view(np.uint64)

    def empty_u64(self, *shape):
        return self.torch.empty(shape, dtype=self.torch.int64, device=self.dev)

    def load_keys(self, keys: dict, extra_steps=()):
        """keys: {galois element: array [r][2][r+1][N]} from the oracle, plus the rotation amounts."""
        steps = list(ckks.required_rotations(self.plan)) + list(extra_steps)
        uniq = []
        for s in steps:
            if s % self.par.n and s % self.par.n not in uniq:
                uniq.append(s % self.par.n)
        if not uniq:                     # a plan with a single diagonal per tile needs no rotation
            return uniq
        arr = np.stack([keys[ckks.galois_element(s, self.par.N)] for s in uniq])
        self.bf.bf_load_eval_keys(self.ctx, uniq, len(uniq), self.to_dev(arr))
        return uniq

    def linear(self, cts, W, d_out, d_in, weights=None):
        n_in, n_out = len(cts), self.plan.n_out(d_out)
        ct_in = self.to_dev(np.stack(cts))
        ct_out = self.empty_u64(n_out, 2, self.par.r, self.par.N)
        Wd = self.to_dev(np.ascontiguousarray(W, dtype=np.float32))
        self.bf.bf_linear(self.ctx, ct_in, n_in, weights, None if weights is not None else Wd, d_out, d_in,
                          ct_out, n_out)
        return ct_out
