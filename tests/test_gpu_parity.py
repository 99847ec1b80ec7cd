"""GPU parity: every kernel family and every entry point of the C ABI against the CPU oracle,
bit for bit on every residue, on the same seeded inputs."""
import numpy as np
import pytest

from oracle import ckks
from paper_2606_17421_b200 import workloads as wl
from tests.helpers import GpuSide, custom_params, oracle_params

pytestmark = pytest.mark.gpu

# the plan variant the benchmark's headline runs: two row blocks per plaintext, one division by P per output
# ciphertext, baby-step rotations kept in the extended basis
BEST = dict(pack="complex", moddown="per_output", hoist="double")


# ------------------------------------------------------------------ transforms

@pytest.mark.parametrize("logN,n_small", [(10, 1), (12, 2), (13, 3), (15, 6), (16, 8)])
def test_negacyclic_mul_matches_oracle(logN, n_small):
    N = 1 << logN
    par = custom_params(N, n_small)
    g = GpuSide(par, ckks.Plan(64, 1, 8, 8))
    try:
        nb = par.r + 1
        n_polys = 2 * nb + 3                      # not a whole number of basis groups
        rng = np.random.default_rng(logN)
        moduli = [par.basis[t % nb] for t in range(n_polys)]
        a = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
        b = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
        a[0, :] = np.uint64(moduli[0] - 1)        # extreme residues
        b[0, :] = np.uint64(moduli[0] - 1)
        a[1, :] = 0
        out = g.empty_u64(n_polys, N)
        g.bf.bf_negacyclic_mul(g.ctx, g.to_dev(a), g.to_dev(b), out, n_polys)
        expect = ckks.ring_mul(a, b, moduli, par)
        assert np.array_equal(g.to_host_u64(out), expect)
    finally:
        g.close()


# ------------------------------------------------------------------ encoder

ENCODE_CASES = [
    # param set / ring, plan, (d_out, d_in)
    ("n12", (64, 1, 8, 8), (64, 64)),
    ("n12", (64, 4, 4, 4), (100, 130)),          # ragged: zero padding in rows and columns
    ("n12", (256, 8, 8, 4), (300, 256)),
    ("n15", (1024, 16, 8, 8), (1100, 768)),
]


@pytest.mark.parametrize("compact", [False, True])
@pytest.mark.parametrize("pack", ["real", "complex"])
@pytest.mark.parametrize("pkey,plan_t,shape", ENCODE_CASES)
def test_encode_weights_matches_oracle(pkey, plan_t, shape, compact, pack):
    par = oracle_params(pkey)
    plan = ckks.Plan(*plan_t, pack=pack)
    d_out, d_in = shape
    W = wl.gen_weights(1, f"enc{pkey}{plan_t}", d_out, d_in)
    g = GpuSide(par, plan)
    try:
        g.bf.bf_set_compact_cache(g.ctx, compact)
        w = g.bf.bf_encode_weights(g.ctx, g.to_dev(W), d_out, d_in)
        n_in, n_out = -(-d_in // plan.D), plan.n_out(d_out)
        used = g.bf.bf_cache_bytes_used(g.ctx)
        assert used == g.bf.bf_weights_bytes(g.ctx, d_out, d_in)
        # every encoded word is resident once: 8 bytes, or in the compact cache the narrowest format its
        # prime allows (4, 5 or 8 bytes); layout padding comes on top
        word_bytes = sum(4 if q < 2 ** 32 else 5 if q < 2 ** 40 else 8 for q in par.primes) if compact else 8 * par.r
        words = n_in * n_out * plan.M * par.N
        assert words * word_bytes <= used
        if compact and word_bytes < 8 * par.r:
            g.bf.bf_set_compact_cache(g.ctx, False)
            assert used < g.bf.bf_weights_bytes(g.ctx, d_out, d_in)
            g.bf.bf_set_compact_cache(g.ctx, True)
        idx = [(p, q, j, k) for p in range(n_out) for q in range(n_in) for j in range(plan.g) for k in range(plan.b)]
        if len(idx) > 48:                         # sample, always keeping the corners
            rng = np.random.default_rng(0)
            keep = {0, len(idx) - 1} | set(rng.choice(len(idx), 46, replace=False).tolist())
            idx = [idx[i] for i in sorted(keep)]
        out = g.empty_u64(par.r, par.N)
        for (p, q, j, k) in idx:
            z = ckks.plain_slots(W, plan, p, q, j, k, par.n)
            expect = ckks.to_residues(ckks.encode_coeffs(z, par.N, par.scale), par.primes)
            g.bf.bf_weights_export(g.ctx, w, p, q, j, k, out)
            assert np.array_equal(g.to_host_u64(out), expect), (p, q, j, k)
        g.bf.bf_weights_free(g.ctx, w)
        assert g.bf.bf_cache_bytes_used(g.ctx) == 0
    finally:
        g.close()


# ------------------------------------------------------------------ key switch, rescale

@pytest.mark.parametrize("pkey", ["n12", "n15"])
def test_rotate_matches_oracle(pkey):
    par = oracle_params(pkey)
    plan = ckks.Plan(64, 1, 8, 8) if pkey == "n12" else ckks.Plan(1024, 16, 4, 16)
    s = ckks.keygen(par, 3)
    keys = ckks.make_rotation_keys(par, s, plan, 3)
    g = GpuSide(par, plan)
    try:
        steps = g.load_keys(keys)
        rng = np.random.default_rng(7)
        z = rng.normal(size=par.n)
        ct = ckks.encrypt(par, s, ckks.encode_coeffs(z, par.N, par.scale), 4)
        out = g.empty_u64(2, par.r, par.N)
        for st in steps[:4] + steps[-2:]:
            g.bf.bf_rotate(g.ctx, g.to_dev(ct), st, out)
            expect = ckks.rotate(par, ct, st, keys)
            got = g.to_host_u64(out)
            assert np.array_equal(got, expect), st
            dec = ckks.decode(ckks.decrypt(par, s, got), par.N, par.scale)
            assert np.abs(dec - np.roll(z, -st)).max() < 1e-6
        with pytest.raises(g.bf.BifrostError) as ei:
            g.bf.bf_rotate(g.ctx, g.to_dev(ct), 12345, out)
        assert ei.value.code == g.bf.BF_ERR_MISSING_KEY
    finally:
        g.close()


@pytest.mark.parametrize("pkey", ["n12", "n15"])
def test_rescale_matches_oracle(pkey):
    par = oracle_params(pkey)
    g = GpuSide(par, ckks.Plan(64, 1, 8, 8))
    try:
        rng = np.random.default_rng(8)
        cts = np.stack([np.stack([ckks.sample_uniform(rng, par.primes, par.N) for _ in range(2)]) for _ in range(3)])
        cts[0, 0, -1, :5] = [0, 1, (par.primes[-1] - 1) // 2, (par.primes[-1] - 1) // 2 + 1, par.primes[-1] - 1]
        expect = np.stack([ckks.rescale(par, c) for c in cts])
        d_in = g.to_dev(cts)
        d_out = g.empty_u64(3, 2, par.r - 1, par.N)
        new_scale = g.bf.bf_rescale(g.ctx, d_in, d_out, 3, par.r, par.scale * par.scale)
        assert np.array_equal(g.to_host_u64(d_out), expect)
        assert new_scale == par.scale * par.scale / par.primes[-1]
        # in place, several ciphertexts
        g.bf.bf_rescale(g.ctx, d_in, d_in, 3, par.r)
        flat = g.to_host_u64(d_in).reshape(-1)[:expect.size].reshape(expect.shape)
        assert np.array_equal(flat, expect)
        # a second level down, from the packed output
        expect2 = np.stack([ckks.rescale(par, c) for c in expect])
        d2 = g.empty_u64(3, 2, par.r - 2, par.N)
        if par.r - 1 >= 2:
            g.bf.bf_rescale(g.ctx, d_out, d2, 3, par.r - 1)
            assert np.array_equal(g.to_host_u64(d2), expect2)
        with pytest.raises(g.bf.BifrostError) as ei:
            g.bf.bf_rescale(g.ctx, d_in, d_in, 1, 1)
        assert ei.value.code == g.bf.BF_ERR_LEVEL
    finally:
        g.close()


# ------------------------------------------------------------------ the linear layer

def run_case(par, plan, d_out, d_in, seed, tol, tag, tight=1e-5):
    W = wl.gen_weights(seed, tag, d_out, d_in)
    x = wl.gen_activation(seed, tag, d_in)
    s = ckks.keygen(par, seed)
    keys = ckks.make_rotation_keys(par, s, plan, seed)
    cts = ckks.encrypt_vector(par, plan, s, x, seed)
    expect = ckks.linear(par, plan, cts, W, keys)
    n_out = plan.n_out(d_out)
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        Wd = g.to_dev(W)
        w = g.bf.bf_encode_weights(g.ctx, Wd, d_out, d_in)
        got_cached = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=w))
        got_fallback = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=None))
        for p in range(n_out):
            assert np.array_equal(got_cached[p], expect[p]), ("cached", p)
            assert np.array_equal(got_fallback[p], expect[p]), ("fallback", p)
        # the configuration the benchmark times: the same buffers again and again, so that the call is
        # captured and then replayed as a graph with its concurrent key-switch lanes
        ct_in = g.to_dev(np.stack(cts))
        ct_out = g.empty_u64(n_out, 2, par.r, par.N)
        for call in range(4):
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, len(cts), w, None, d_out, d_in, ct_out, n_out)
        got_replayed = g.to_host_u64(ct_out)
        for p in range(n_out):
            assert np.array_equal(got_replayed[p], expect[p]), ("replayed", p)
        # the compact cache format (narrower words per prime) changes no residue, cached or on the fly
        g.bf.bf_set_compact_cache(g.ctx, True)
        w_compact = g.bf.bf_encode_weights(g.ctx, Wd, d_out, d_in)
        got_compact = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=w_compact))
        got_compact_fallback = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=None))
        got_mixed = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=w))        # the older handle still works
        g.bf.bf_set_compact_cache(g.ctx, False)
        for p in range(n_out):
            assert np.array_equal(got_compact[p], expect[p]), ("compact", p)
            assert np.array_equal(got_compact_fallback[p], expect[p]), ("compact fallback", p)
            assert np.array_equal(got_mixed[p], expect[p]), ("mixed", p)
        g.bf.bf_weights_free(g.ctx, w_compact)
        # rescale on the device, decrypt on the host, compare with the fp64 product
        d_ct = g.to_dev(got_cached)
        low = g.empty_u64(n_out, 2, par.r - 1, par.N)
        scale = g.bf.bf_rescale(g.ctx, d_ct, low, n_out, par.r, par.scale * par.scale)
        low = g.to_host_u64(low)
        y = np.zeros(d_out)
        for p in range(n_out):
            assert np.array_equal(low[p], ckks.rescale(par, expect[p]))
            part = ckks.fold_output(ckks.decode(ckks.decrypt(par, s, low[p]), par.N, scale), plan, p, d_out)
            y[p * plan.rows_per_ct:p * plan.rows_per_ct + len(part)] = part
        err = np.abs(y - W.astype(np.float64) @ x).max()
        assert err < tol, err
        assert err < tight         # far inside the stated tolerance; catches scale bookkeeping slips
        # the host-buffer entry point gives the same rescaled ciphertexts
        import torch
        h_in = torch.from_numpy(np.stack(cts).view(np.int64)).pin_memory()
        h_out = torch.empty((n_out, 2, par.r - 1, par.N), dtype=torch.int64).pin_memory()
        g.bf.bf_linear_host(g.ctx, h_in, len(cts), w, None, d_out, d_in, h_out, n_out)
        assert np.array_equal(h_out.numpy().view(np.uint64), low)
        # product and rescale as one call: cached (direct, captured, replayed) and on the fly
        low_fused = g.empty_u64(n_out, 2, par.r - 1, par.N)
        for call in range(3):
            low_fused.zero_()
            assert g.bf.bf_linear_rescaled(g.ctx, ct_in, len(cts), w, None, d_out, d_in, low_fused, n_out,
                                           par.scale * par.scale) == scale
        assert np.array_equal(g.to_host_u64(low_fused), low)
        low_fused.zero_()
        g.bf.bf_linear_rescaled(g.ctx, ct_in, len(cts), None, Wd, d_out, d_in, low_fused, n_out)
        assert np.array_equal(g.to_host_u64(low_fused), low)
        # the two entry points on the SAME output address (replayed launch sequences are keyed by the arguments):
        # a full-level result, then a rescaled one, then a full-level one again, each repeated into its replay
        shared = g.empty_u64(n_out, 2, par.r, par.N)
        shared_low = shared.view(-1)[:n_out * 2 * (par.r - 1) * par.N].view(n_out, 2, par.r - 1, par.N)
        for kind in ("full", "rescaled", "full"):
            for call in range(3):
                shared.zero_()
                if kind == "full":
                    g.bf.bf_linear(g.ctx, ct_in, len(cts), w, None, d_out, d_in, shared, n_out)
                else:
                    g.bf.bf_linear_rescaled(g.ctx, ct_in, len(cts), w, None, d_out, d_in, shared_low, n_out)
            if kind == "full":
                assert np.array_equal(g.to_host_u64(shared), got_cached), kind
            else:
                assert np.array_equal(g.to_host_u64(shared_low), low), kind
    finally:
        g.close()


def test_linear_tiny_config_bit_exact():
    w = wl.WORKLOADS["tiny"]
    par = oracle_params(w.params)
    run_case(par, ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g), 64, 64, 0, 1e-2, "tiny")


@pytest.mark.parametrize("plan_t,shape", [
    ((64, 4, 4, 4), (100, 130)),      # tau > 1, ragged rows and columns, 2 x 3 tiles
    ((64, 32, 2, 1), (64, 64)),       # fully dense packing, no giant step
    ((128, 1, 1, 128), (128, 128)),   # no baby step: every diagonal its own giant rotation
    ((32, 1, 32, 1), (40, 32)),       # all rotations hoisted from the input
    ((32, 32, 1, 1), (70, 50)),       # one diagonal per tile: no rotation at all, 3 x 2 tiles
    ((64, 4, 16, 1), (150, 64)),      # 16 terms per output group, odd number of groups: half-filled last stage
    ((64, 4, 4, 4), (64, 1472)),      # 23 input chunks: their 69 baby rotations span two key-switch batches
    ((64, 4, 4, 4), (1920, 64)),      # 30 output blocks: their 90 giant rotations span two key-switch batches
])
def test_linear_small_ring_plans(plan_t, shape):
    par = oracle_params("n12")
    run_case(par, ckks.Plan(*plan_t), shape[0], shape[1], 2, 1e-2, f"small{plan_t}")


@pytest.mark.parametrize("plan_t,shape", [
    ((64, 4, 4, 4), (100, 130)),      # two row blocks -> one output ciphertext, ragged second block
    ((64, 4, 4, 4), (150, 64)),       # three row blocks -> two ciphertexts, the last one with an empty imaginary part
    ((64, 1, 8, 8), (128, 64)),       # classical replicated layout, both parts full
    ((32, 32, 1, 1), (70, 50)),       # no rotation at all
    ((64, 4, 4, 4), (1920, 64)),      # 15 output ciphertexts
])
def test_linear_complex_packing_small_ring(plan_t, shape):
    par = oracle_params("n12")
    run_case(par, ckks.Plan(*plan_t, pack="complex"), shape[0], shape[1], 6, 1e-2, f"cplx{plan_t}")


def test_linear_gpt2_qkv_complex_packing_bit_exact():
    # the 768 -> 2304 projection with two row blocks per plaintext: 2 output ciphertexts instead of 3
    w = wl.WORKLOADS["gpt2_qkv"]
    par = oracle_params(w.params)
    L = w.layers[0]
    run_case(par, ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, pack="complex"), L.d_out, L.d_in, 0, 1e-3, L.name)


@pytest.mark.parametrize("pack", ["real", "complex"])
@pytest.mark.parametrize("plan_t,shape", [
    ((64, 4, 4, 4), (100, 130)),      # three giant rotations per output, two or one output ciphertexts
    ((64, 1, 8, 8), (128, 64)),       # seven giant rotations per output
    ((64, 1, 2, 32), (64, 64)),       # 31 giant rotations summed before the one division
    ((64, 32, 2, 1), (64, 64)),       # no giant step: nothing to merge
    ((64, 4, 4, 4), (1920, 64)),      # 90 (45) giant rotations: several key-switch launches feed one division stage
])
def test_linear_one_division_by_P_per_output_small_ring(plan_t, shape, pack):
    par = oracle_params("n12")
    run_case(par, ckks.Plan(*plan_t, pack=pack, moddown="per_output"), shape[0], shape[1], 7, 1e-2, f"po{plan_t}")


@pytest.mark.parametrize("pack", ["real", "complex"])
def test_linear_gpt2_qkv_one_division_by_P_per_output_bit_exact(pack):
    w = wl.WORKLOADS["gpt2_qkv"]
    par = oracle_params(w.params)
    L = w.layers[0]
    plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, pack=pack, moddown="per_output")
    run_case(par, plan, L.d_out, L.d_in, 0, 1e-3, L.name)


@pytest.mark.parametrize("pack,moddown", [("real", "per_rotation"), ("complex", "per_output")])
@pytest.mark.parametrize("plan_t,shape", [
    ((64, 4, 4, 4), (100, 130)),      # three input ciphertexts, ragged
    ((64, 1, 8, 8), (128, 64)),       # classical layout, seven baby rotations
    ((64, 32, 2, 1), (64, 64)),       # no giant step
    ((128, 1, 1, 128), (128, 128)),   # no baby step: only P * ct, whose division by P is exact
    ((64, 4, 16, 1), (150, 64)),      # 16 terms per group, half-filled last stage
    ((64, 4, 4, 4), (64, 1472)),      # 23 input ciphertexts: their baby rotations span two key-switch batches
])
def test_linear_double_hoisting_small_ring(plan_t, shape, pack, moddown):
    if plan_t[3] - 1 > 64 and moddown == "per_output":
        pytest.skip("per-output division sums at most 64 giant steps")
    par = oracle_params("n12")
    run_case(par, ckks.Plan(*plan_t, pack=pack, moddown=moddown, hoist="double"), shape[0], shape[1], 8, 1e-2, f"dh{plan_t}")


@pytest.mark.parametrize("pack,moddown", [("real", "per_rotation"), ("complex", "per_output")])
def test_linear_gpt2_qkv_double_hoisting_bit_exact(pack, moddown):
    w = wl.WORKLOADS["gpt2_qkv"]
    par = oracle_params(w.params)
    L = w.layers[0]
    plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, pack=pack, moddown=moddown, hoist="double")
    run_case(par, plan, L.d_out, L.d_in, 0, 1e-3, L.name)


def test_linear_double_hoisting_with_the_papers_own_parameter_set():
    # a 60-bit ciphertext prime next to the 60-bit special prime: whole-word accumulation for every prime
    par = oracle_params("paper_n13")
    run_case(par, ckks.Plan(256, 16, 4, 4, hoist="double"), 300, 520, 4, 1e-2, "paper_n13_dh", tight=1e-3)


@pytest.mark.parametrize("bits", [64, 32])
@pytest.mark.parametrize("modes", [{}, BEST], ids=["plain", "best"])
def test_weights_kept_as_coefficients_give_the_same_ciphertexts(bits, modes):
    # the coefficient form of the cache: rounded integer coefficients are resident, reduced per prime and
    # transformed on every call; residues must not change, and the handle is 1/r (1/2r) of the usual size
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4, **modes)
    d_out, d_in = 150, 130
    s = ckks.keygen(par, 61)
    keys = ckks.make_rotation_keys(par, s, plan, 61)
    W = wl.gen_weights(61, "coef", d_out, d_in)
    if bits == 32:      # on this small ring the slot vectors repeat eight times, which concentrates the coefficients:
        W = W / 32      # keep them inside 32 bits (the full-size rings have no replication and fit as they are)
    cts = ckks.encrypt_vector(par, plan, s, wl.gen_activation(61, "coef", d_in), 61)
    expect = ckks.linear(par, plan, cts, W, keys)
    n_out, n_in = plan.n_out(d_out), 3
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        Wd = g.to_dev(W)
        full_bytes = g.bf.bf_weights_bytes(g.ctx, d_out, d_in)
        g.bf.bf_set_coefficient_cache(g.ctx, bits)
        w = g.bf.bf_encode_weights(g.ctx, Wd, d_out, d_in)
        used = g.bf.bf_cache_bytes_used(g.ctx)
        assert used == n_in * n_out * plan.M * par.N * bits // 8 == g.bf.bf_weights_bytes(g.ctx, d_out, d_in)
        assert used * par.r * (64 // bits) <= full_bytes
        ct_in = g.to_dev(np.stack(cts))
        ct_out = g.empty_u64(n_out, 2, par.r, par.N)
        for call in range(4):                       # direct, captured, replayed
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, n_in, w, None, d_out, d_in, ct_out, n_out)
            got = g.to_host_u64(ct_out)
            for p in range(n_out):
                assert np.array_equal(got[p], expect[p]), (call, p)
        out = g.empty_u64(par.r, par.N)
        for (p, q, j, k) in ((0, 0, 0, 0), (n_out - 1, 2, 3, 1), (0, 1, 2, 3)):
            z = ckks.plain_slots(W, plan, p, q, j, k, par.n)
            g.bf.bf_weights_export(g.ctx, w, p, q, j, k, out)
            assert np.array_equal(g.to_host_u64(out), ckks.to_residues(ckks.encode_coeffs(z, par.N, par.scale), par.primes))
        # a transform-domain handle made afterwards works beside it
        g.bf.bf_set_coefficient_cache(g.ctx, 0)
        w2 = g.bf.bf_encode_weights(g.ctx, Wd, d_out, d_in)
        got = g.to_host_u64(g.linear(cts, W, d_out, d_in, weights=w2))
        assert all(np.array_equal(got[p], expect[p]) for p in range(n_out))
        g.bf.bf_weights_free(g.ctx, w)
        g.bf.bf_weights_free(g.ctx, w2)
        assert g.bf.bf_cache_bytes_used(g.ctx) == 0
        if bits == 32:      # coefficients beyond 32 bits are refused at encoding time
            g.bf.bf_set_coefficient_cache(g.ctx, 32)
            with pytest.raises(g.bf.BifrostError) as ei:
                g.bf.bf_encode_weights(g.ctx, g.to_dev(W * 1024), d_out, d_in)
            assert ei.value.code == g.bf.BF_ERR_RANGE
            assert g.bf.bf_cache_bytes_used(g.ctx) == 0
        with pytest.raises(g.bf.BifrostError):
            g.bf.bf_set_coefficient_cache(g.ctx, 16)
    finally:
        g.close()


def test_per_output_division_refuses_more_giant_steps_than_it_can_sum():
    from paper_2606_17421_b200 import bifrost as bf
    ps = wl.PARAM_SETS["n12"]
    basis = list(ps["primes"]) + [ps["special"]]
    with pytest.raises(bf.BifrostError) as ei:          # g - 1 = 127 > 64
        bf.bf_ctx_create(ps["N"], basis, 3, 2.0 ** 40, bf.bf_plan(128, 1, 1, 128, bf.BF_PLAN_MODDOWN_PER_OUTPUT))
    assert ei.value.code == bf.BF_ERR_SHAPE
    with pytest.raises(bf.BifrostError) as ei:          # unknown flag bit
        bf.bf_ctx_create(ps["N"], basis, 3, 2.0 ** 40, bf.bf_plan(64, 1, 8, 8, 64))
    assert ei.value.code == bf.BF_ERR_INVALID_ARG


@pytest.mark.parametrize("modes", [{}, BEST, dict(hoist="double")], ids=["plain", "best", "double_hoist"])
def test_weights_with_a_split_of_their_own(modes):
    # one context (plan 8 x 4), three handles for the same matrix with the splits 8 x 4, 16 x 2 and 2 x 16, and a
    # coefficient-form handle with 4 x 8: every call matches the oracle run under that split; what the context
    # refuses: a split whose product is not D / tau, one that is not a power of two, a missing key
    from paper_2606_17421_b200 import bifrost as bf
    par = oracle_params("n12")
    base = ckks.Plan(64, 2, 8, 4, **modes)
    d_out, d_in, seed = 150, 100, 21
    W = wl.gen_weights(seed, "split", d_out, d_in)
    x = wl.gen_activation(seed, "split", d_in)
    s = ckks.keygen(par, seed)
    variants = [(8, 4), (16, 2), (2, 16), (4, 8)]
    plans = [ckks.Plan(base.D, base.tau, b, g, base.pack, base.moddown, base.hoist) for b, g in variants]
    extra = sorted({st for pl in plans for st in ckks.required_rotations(pl)})
    keys = ckks.make_rotation_keys(par, s, base, seed, extra_steps=extra)
    cts = ckks.encrypt_vector(par, base, s, x, seed)
    g = GpuSide(par, base)
    try:
        Wd = g.to_dev(W)
        g.load_keys(keys)                            # the keys of the plan's own split only
        w = g.bf.bf_encode_weights_split(g.ctx, Wd, d_out, d_in, 16, 2)
        with pytest.raises(bf.BifrostError) as ei:
            g.linear(cts, W, d_out, d_in, weights=w)
        assert ei.value.code == bf.BF_ERR_MISSING_KEY
        g.bf.bf_weights_free(g.ctx, w)
        g.load_keys(keys, extra_steps=extra)
        for bad in ((8, 8), (3, 11), (0, 32), (32, 0)):
            with pytest.raises(bf.BifrostError) as ei:
                g.bf.bf_encode_weights_split(g.ctx, Wd, d_out, d_in, *bad)
            assert ei.value.code == bf.BF_ERR_SHAPE, bad
        for (b, gg), plan in zip(variants, plans):
            expect = ckks.linear(par, plan, cts, W, keys)
            if (b, gg) == (4, 8):
                g.bf.bf_set_coefficient_cache(g.ctx, 64)
            w = g.bf.bf_encode_weights_split(g.ctx, Wd, d_out, d_in, b, gg)
            g.bf.bf_set_coefficient_cache(g.ctx, 0)
            n_out = plan.n_out(d_out)
            ct_in = g.to_dev(np.stack(cts))
            out = g.empty_u64(n_out, 2, par.r, par.N)
            for call in range(3):               # direct, captured, replayed
                out.zero_()
                g.bf.bf_linear(g.ctx, ct_in, len(cts), w, None, d_out, d_in, out, n_out)
            got = g.to_host_u64(out)
            for p in range(n_out):
                assert np.array_equal(got[p], expect[p]), (b, gg, p)
            g.bf.bf_weights_free(g.ctx, w)
    finally:
        g.close()


@pytest.mark.parametrize("case", range(32))
def test_random_small_ring_cases(case):
    # seeded random draws over what the other cases fix by hand: tile side, replica split, baby/giant split of the plan
    # and of the handle, the three plan flags, ragged shapes with one to three input and output blocks; the cached
    # call, the replayed call and the fused product + rescale must all match the oracle
    rng = np.random.default_rng(1000 + case)
    par = oracle_params("n12")
    D = int(rng.choice([32, 64, 128]))
    tau = int(rng.choice([t for t in (1, 2, 4, 8, 16) if D * t <= par.n and D // t >= 2]))
    M = D // tau
    splits = [(b, M // b) for b in (1, 2, 4, 8, 16, 32, 64) if b <= M and M % b == 0 and b - 1 <= 64 and M // b - 1 <= 64]
    b, g_ = splits[int(rng.integers(len(splits)))]
    hb, hg = splits[int(rng.integers(len(splits)))]
    modes = dict(pack=str(rng.choice(["real", "complex"])), moddown=str(rng.choice(["per_rotation", "per_output"])),
                 hoist=str(rng.choice(["single", "double"])))
    d_in = int(rng.integers(1, 3 * D + 1))
    d_out = int(rng.integers(1, 3 * D + 1))
    base = ckks.Plan(D, tau, b, g_, **modes)
    hplan = ckks.Plan(D, tau, hb, hg, **modes)
    seed = 2000 + case
    W = wl.gen_weights(seed, "rand", d_out, d_in)
    x = wl.gen_activation(seed, "rand", d_in)
    s = ckks.keygen(par, seed)
    extra = ckks.required_rotations(hplan)
    keys = ckks.make_rotation_keys(par, s, base, seed, extra_steps=extra)
    cts = ckks.encrypt_vector(par, base, s, x, seed)
    expect_base = ckks.linear(par, base, cts, W, keys)
    expect_h = ckks.linear(par, hplan, cts, W, keys)
    n_out = base.n_out(d_out)
    g = GpuSide(par, base)
    try:
        g.load_keys(keys, extra_steps=extra)
        Wd = g.to_dev(W)
        ct_in = g.to_dev(np.stack(cts))
        for plan, expect, w in ((base, expect_base, g.bf.bf_encode_weights(g.ctx, Wd, d_out, d_in)),
                                (hplan, expect_h, g.bf.bf_encode_weights_split(g.ctx, Wd, d_out, d_in, hb, hg))):
            out = g.empty_u64(n_out, 2, par.r, par.N)
            low = g.empty_u64(n_out, 2, par.r - 1, par.N)
            for call in range(3):
                out.zero_()
                low.zero_()
                g.bf.bf_linear(g.ctx, ct_in, len(cts), w, None, d_out, d_in, out, n_out)
                g.bf.bf_linear_rescaled(g.ctx, ct_in, len(cts), w, None, d_out, d_in, low, n_out)
            got, got_low = g.to_host_u64(out), g.to_host_u64(low)
            for p in range(n_out):
                assert np.array_equal(got[p], expect[p]), (case, plan, p)
                assert np.array_equal(got_low[p], ckks.rescale(par, expect[p])), (case, plan, p, "rescaled")
            g.bf.bf_weights_free(g.ctx, w)
        fly = g.to_host_u64(g.linear(cts, W, d_out, d_in))          # on the fly: the plan's own split
        for p in range(n_out):
            assert np.array_equal(fly[p], expect_base[p]), (case, p, "on the fly")
    finally:
        g.close()


def test_linear_gpt2_qkv_config_bit_exact():
    w = wl.WORKLOADS["gpt2_qkv"]
    par = oracle_params(w.params)
    L = w.layers[0]
    run_case(par, ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g), L.d_out, L.d_in, 0, 1e-3, L.name)


def check_blocks(par, plan, layers, blocks_of, seed, on_the_fly=(), splits=None):
    """Full-size calls exactly as the benchmark's runner issues them (projections that read the same
    activation stacked row-wise into one call, repeated on the same buffers so that the third call is the
    replayed graph with its concurrent key-switch chains): the device computes every output block, the
    oracle the listed ones; those must agree on every residue, before and after the rescale, and decrypt
    to the fp64 product.  Calls with the same d_in share one set of input ciphertexts, so that the
    oracle rotates them only once.  splits: {call name: (b, g)}, the calls whose weights are encoded with a
    baby/giant split of their own (as the runner does under the headline plan)."""
    splits = splits or {}
    assert not set(splits) & set(on_the_fly)        # the on-the-fly path runs under the plan's own split
    base = plan
    plans = {name: ckks.Plan(base.D, base.tau, b, g, base.pack, base.moddown, base.hoist) for name, (b, g) in splits.items()}
    extra = sorted({st for pl in plans.values() for st in ckks.required_rotations(pl)})
    s = ckks.keygen(par, seed)
    keys = ckks.make_rotation_keys(par, s, base, seed, extra_steps=extra)
    units = wl.fuse_shared_inputs(layers, base.D)
    inputs, rotated = {}, {}         # d_in -> (x, ciphertexts); (d_in, b) -> the oracle's baby rotations
    g = GpuSide(par, base)
    try:
        g.load_keys(keys, extra_steps=extra)
        for name, d_in, members in units:
            plan = plans.get(name, base)
            d_out = sum(m.d_out for m in members)
            W = np.concatenate([wl.gen_weights(seed, m.name, m.d_out, m.d_in) for m in members], axis=0)
            if d_in not in inputs:
                x = wl.gen_activation(seed, f"x{d_in}", d_in)
                inputs[d_in] = (x, ckks.encrypt_vector(par, base, s, x, seed))
            x, cts = inputs[d_in]
            if (d_in, plan.b) not in rotated:
                rot_fn = ckks.baby_rotations_ext if plan.hoist == "double" else ckks.baby_rotations
                rotated[(d_in, plan.b)] = [rot_fn(par, plan, ct, keys) for ct in cts]
            X = rotated[(d_in, plan.b)]
            n_in, n_out = len(cts), plan.n_out(d_out)
            blocks = list(blocks_of(name, n_out))
            expect = ckks.linear(par, plan, cts, W, keys, blocks=blocks, X=X)
            if name in splits:
                w = g.bf.bf_encode_weights_split(g.ctx, g.to_dev(W), d_out, d_in, plan.b, plan.g)
            else:
                w = g.bf.bf_encode_weights(g.ctx, g.to_dev(W), d_out, d_in)
            ct_in = g.to_dev(np.stack(cts))
            out = g.empty_u64(n_out, 2, par.r, par.N)
            for call in range(3):               # direct, captured, replayed
                out.zero_()
                g.bf.bf_linear(g.ctx, ct_in, n_in, w, None, d_out, d_in, out, n_out)
            if name in on_the_fly:          # the same call with the weights encoded on the fly
                fly = g.to_host_u64(g.linear(cts, W, d_out, d_in))
                for p in blocks:
                    assert np.array_equal(fly[p], expect[p]), (name, p, "on the fly")
                del fly
            low = g.empty_u64(n_out, 2, par.r - 1, par.N)
            scale = g.bf.bf_rescale(g.ctx, out, low, n_out, par.r, par.scale * par.scale)
            # the call the runner makes: product and rescale in one (direct, captured, replayed)
            low_fused = g.empty_u64(n_out, 2, par.r - 1, par.N)
            for call in range(3):
                low_fused.zero_()
                scale_fused = g.bf.bf_linear_rescaled(g.ctx, ct_in, n_in, w, None, d_out, d_in, low_fused, n_out,
                                                      par.scale * par.scale)
            assert scale_fused == scale
            got, low, low_fused = g.to_host_u64(out), g.to_host_u64(low), g.to_host_u64(low_fused)
            assert np.array_equal(low_fused, low), name       # every output ciphertext
            g.bf.bf_weights_free(g.ctx, w)
            y_ref = W.astype(np.float64) @ x
            for p in blocks:
                assert np.array_equal(got[p], expect[p]), (name, p)
                assert np.array_equal(low[p], ckks.rescale(par, expect[p])), (name, p)
                part = ckks.fold_output(ckks.decode(ckks.decrypt(par, s, low[p]), par.N, scale), plan, p, d_out)
                err = np.abs(part - y_ref[p * plan.rows_per_ct:p * plan.rows_per_ct + len(part)]).max()
                assert err < 1e-3, (name, p, err)
    finally:
        g.close()


@pytest.mark.parametrize("modes", [{}, BEST], ids=["plain", "best"])
def test_gpt2_step_one_whole_layer_every_block(modes):
    # config 2: one transformer layer of the GPT-2 decode step, all four calls, every output ciphertext
    # (qkv 3 row blocks, out_proj 1, ffn_up 3, ffn_down 1 with three input ciphertexts)
    w = wl.WORKLOADS["gpt2_step"]
    par = oracle_params(w.params)
    plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, **modes)
    check_blocks(par, plan, w.layers, lambda name, n_out: range(n_out), 11, splits=w.splits if modes else None)


@pytest.mark.parametrize("modes", [{}, BEST], ids=["plain", "best"])
def test_qwen3_step_the_calls_of_one_layer(modes):
    # config 3: the four calls the runner issues per layer.  q+k+v (1024 -> 4096) in full; o (2048 -> 1024, two
    # input ciphertexts) in full, also on the fly; gate+up (1024 -> 6144): its 18 giant rotations run as two
    # chains of 9 -- blocks 0 and 2 lie in the first chain for j = 1, 2 and in the second for j = 3, blocks 3
    # and 5 in the first for j = 1 and in the second for j = 2, 3; down (3072 -> 1024) in full.  With two row
    # blocks per ciphertext: every output ciphertext of every call
    w = wl.WORKLOADS["qwen3_step"]
    par = oracle_params(w.params)
    plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, **modes)
    pick = {"q+k+v": [0, 1, 2, 3], "o": [0], "gate+up": [0, 2, 3, 5], "down": [0]}
    blocks_of = (lambda name, n_out: range(n_out)) if modes else (lambda name, n_out: pick[name])
    check_blocks(par, plan, w.layers, blocks_of, 12, on_the_fly=("o",), splits=w.splits if modes else None)


@pytest.mark.parametrize("modes", [{}, BEST], ids=["plain", "best"])
def test_llama3_layer_the_calls_the_benchmark_times(modes):
    # config 4 at N = 2^16: q+k+v (4096 -> 6144): first block, the k block and the v block; o (4096 -> 4096):
    # first and last; gate+up (4096 -> 28672): 84 giant rotations in four launches of 22, 22, 22 and 18 --
    # rotation (j - 1) * 28 + p of block p, so block 0 meets launches 1, 2, 3; block 14 (first of up) 1, 2, 4;
    # blocks 21 and 22 the end of launch 1 and the start of launch 2; block 27 launches 2, 3 and the very last
    # rotation; down (14336 -> 4096): 14 input ciphertexts whose 98 baby rotations share two hoisted ModUps
    # (9 + 5 ciphertexts), every output block, and once more with the weights encoded on the fly.
    # With two row blocks per ciphertext gate+up has 14 outputs and 42 giant rotations in launches of 22 and 20:
    # rotation (j - 1) * 14 + p, so ciphertext 0 meets launch 1 twice and launch 2, ciphertexts 7 and 8 the end of
    # launch 1 and the start of launch 2, ciphertext 13 the very last rotation
    w = wl.WORKLOADS["llama3_layer"]
    par = oracle_params(w.params)
    plan = ckks.Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, **modes)
    if modes:
        pick = {"q+k+v": [0, 2], "o": [0, 1], "gate+up": [0, 7, 8, 13], "down": [0, 1]}
    else:
        pick = {"q+k+v": [0, 4, 5], "o": [0, 3], "gate+up": [0, 14, 21, 22, 27], "down": [0, 1, 2, 3]}
    # (under the headline plan gate+up and down run with splits of their own, 16 x 2 and 4 x 8; o is then the call
    # that is also checked with its weights encoded on the fly)
    check_blocks(par, plan, w.layers, lambda name, n_out: pick[name], 13, on_the_fly=("o",) if modes else ("down",),
                 splits=w.splits if modes else None)


def test_linear_with_the_papers_own_parameter_set():
    # N = 8192, primes of [60, 30, 30, 30] bits, scale 2^30, one 60-bit special prime (Sec. 4.2).  The 60-bit
    # ciphertext prime takes the whole-word accumulation paths of the multiply-accumulate and key-switch kernels.
    par = oracle_params("paper_n13")
    run_case(par, ckks.Plan(256, 16, 4, 4), 300, 520, 4, 1e-2, "paper_n13", tight=1e-3)   # scale 2^30: coarser


def test_repeated_calls_replay_a_graph_and_still_read_fresh_inputs():
    # from the third call with the same buffers on, bf_linear replays a captured launch sequence; the
    # data in those buffers may change between calls and results must follow
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4)
    s = ckks.keygen(par, 31)
    keys = ckks.make_rotation_keys(par, s, plan, 31)
    W = wl.gen_weights(31, "graph", 100, 130)
    xs = [wl.gen_activation(31, f"graph{t}", 130) for t in range(2)]
    cts = [ckks.encrypt_vector(par, plan, s, x, 31 + t) for t, x in enumerate(xs)]
    expect = [ckks.linear(par, plan, c, W, keys) for c in cts]
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        w = g.bf.bf_encode_weights(g.ctx, g.to_dev(W), 100, 130)
        ct_in = g.to_dev(np.stack(cts[0]))
        ct_out = g.empty_u64(2, 2, par.r, par.N)
        g.bf.bf_get_kernel_stats(g.ctx)            # reset the launch counters
        for call in range(6):
            which = call % 2
            ct_in.copy_(g.to_dev(np.stack(cts[which])))
            g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
            got = g.to_host_u64(ct_out)
            for p in range(2):
                assert np.array_equal(got[p], expect[which][p]), (call, p)
        stats = g.bf.bf_get_kernel_stats(g.ctx)
        per_call = sum(v[0] for v in stats.values()) / 6
        assert per_call == int(per_call) and per_call > 5       # replays are counted like direct launches
        # turning replay off gives the same results
        g.bf.bf_set_graph_replay(g.ctx, False)
        g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
        assert np.array_equal(g.to_host_u64(ct_out)[0], expect[1][0])
        # plain stream order instead of dependent launches, directly and replayed: same residues
        g.bf.bf_set_dependent_launch(g.ctx, False)
        g.bf.bf_set_graph_replay(g.ctx, True)
        for call in range(4):
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
            got = g.to_host_u64(ct_out)
            for p in range(2):
                assert np.array_equal(got[p], expect[1][p]), (call, p)
        # any number of concurrent key-switch chains, directly and replayed
        g.bf.bf_set_dependent_launch(g.ctx, True)
        for lanes in (1, 3, 4, 2):
            g.bf.bf_set_lanes(g.ctx, lanes)
            for call in range(3):
                ct_out.zero_()
                g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
                got = g.to_host_u64(ct_out)
                for p in range(2):
                    assert np.array_equal(got[p], expect[1][p]), (lanes, call, p)
        # and the just-in-time encoding path under dependent launches
        for call in range(2):
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, 3, None, g.to_dev(W), 100, 130, ct_out, 2)
            got = g.to_host_u64(ct_out)
            for p in range(2):
                assert np.array_equal(got[p], expect[1][p]), (call, p)
    finally:
        g.close()


def test_unloading_keys_invalidates_replayed_launch_sequences():
    # after the keys are dropped, a call that was being replayed from its captured graph must be refused
    # (the graph holds the addresses of the freed key arrays), and reloading the keys must make it work again
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4)
    s = ckks.keygen(par, 51)
    keys = ckks.make_rotation_keys(par, s, plan, 51)
    W = wl.gen_weights(51, "unload", 100, 130)
    cts = ckks.encrypt_vector(par, plan, s, wl.gen_activation(51, "unload", 130), 51)
    expect = ckks.linear(par, plan, cts, W, keys)
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        w = g.bf.bf_encode_weights(g.ctx, g.to_dev(W), 100, 130)
        ct_in = g.to_dev(np.stack(cts))
        ct_out = g.empty_u64(2, 2, par.r, par.N)
        for call in range(4):                       # direct, captured, replayed, replayed
            g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
        assert np.array_equal(g.to_host_u64(ct_out)[1], expect[1])
        g.bf.bf_get_kernel_stats(g.ctx)
        g.bf.bf_load_eval_keys(g.ctx, [], 0, None)
        with pytest.raises(g.bf.BifrostError) as ei:
            g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
        assert ei.value.code == g.bf.BF_ERR_MISSING_KEY
        assert sum(v[0] for v in g.bf.bf_get_kernel_stats(g.ctx).values()) == 0     # nothing was launched
        g.load_keys(keys)
        for call in range(3):
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, 3, w, None, 100, 130, ct_out, 2)
        got = g.to_host_u64(ct_out)
        assert np.array_equal(got[0], expect[0]) and np.array_equal(got[1], expect[1])
    finally:
        g.close()


@pytest.mark.parametrize("modes", [{}, dict(moddown="per_output", hoist="double")], ids=["plain", "extended"])
@pytest.mark.parametrize("lanes", [3, 4])
def test_more_giant_rotations_than_one_launch_holds_with_three_and_four_lanes(lanes, modes):
    # 30 output blocks x 3 giant steps = 90 rotations: as one chain they go in launches of lanes * floor(64 / lanes)
    # rotations, which must not exceed the 64 a launch holds (with 3 lanes: 63); also with the inner sums kept in the
    # extended basis (30 outputs assembled from 90 key-switch results)
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4, **modes)
    d_out, d_in = 1920, 64
    s = ckks.keygen(par, 52)
    keys = ckks.make_rotation_keys(par, s, plan, 52)
    W = wl.gen_weights(52, "lanes", d_out, d_in)
    cts = ckks.encrypt_vector(par, plan, s, wl.gen_activation(52, "lanes", d_in), 52)
    blocks = [0, 20, 21, 29]
    expect = ckks.linear(par, plan, cts, W, keys, blocks=blocks)
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        g.bf.bf_set_lanes(g.ctx, lanes)
        w = g.bf.bf_encode_weights(g.ctx, g.to_dev(W), d_out, d_in)
        ct_in = g.to_dev(np.stack(cts))
        ct_out = g.empty_u64(30, 2, par.r, par.N)
        for call in range(3):                       # direct, captured, replayed
            ct_out.zero_()
            g.bf.bf_linear(g.ctx, ct_in, 1, w, None, d_out, d_in, ct_out, 30)
            got = g.to_host_u64(ct_out)
            for p in blocks:
                assert np.array_equal(got[p], expect[p]), (call, p)
    finally:
        g.close()


@pytest.mark.parametrize("pkey,plan_t,shape", [
    ("n12", (64, 4, 4, 4), (100, 130)),          # tau = 4: rotations by 1 and 2, two output ciphertexts
    ("n12", (32, 32, 1, 1), (70, 50)),           # tau = 32, no other rotation in the plan, three outputs
    ("n15", (1024, 16, 16, 4), (1100, 300)),     # the headline plan: rotations by 1, 2, 4, 8
])
def test_fold_in_ciphertext_matches_oracle(pkey, plan_t, shape):
    par = oracle_params(pkey)
    plan = ckks.Plan(*plan_t)
    d_out, d_in = shape
    s = ckks.keygen(par, 41)
    fold_steps = ckks.fold_rotations(plan)
    keys = ckks.make_rotation_keys(par, s, plan, 41, extra_steps=fold_steps)
    W = wl.gen_weights(41, "fold", d_out, d_in)
    x = wl.gen_activation(41, "fold", d_in)
    cts = ckks.encrypt_vector(par, plan, s, x, 41)
    n_out = -(-d_out // plan.D)
    lin = ckks.linear(par, plan, cts, W, keys)
    expect = [ckks.fold_in_ciphertext(par, plan, lin[p], keys) for p in range(n_out)]
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys, extra_steps=fold_steps)
        out = g.linear(cts, W, d_out, d_in, weights=g.bf.bf_encode_weights(g.ctx, g.to_dev(W), d_out, d_in))
        g.bf.bf_fold(g.ctx, out, n_out)
        got = g.to_host_u64(out)
        for p in range(n_out):
            assert np.array_equal(got[p], expect[p]), p
        # rescale, decrypt: slot (0, kappa, 0) is the complete dot product
        low = g.empty_u64(n_out, 2, par.r - 1, par.N)
        scale = g.bf.bf_rescale(g.ctx, out, low, n_out, par.r, par.scale * par.scale)
        low = g.to_host_u64(low)
        y = np.zeros(d_out)
        for p in range(n_out):
            part = ckks.folded_output(ckks.decode(ckks.decrypt(par, s, low[p]), par.N, scale), plan, p, d_out)
            y[p * plan.D:p * plan.D + len(part)] = part
        assert np.abs(y - W.astype(np.float64) @ x).max() < 1e-3
        # without the keys of the fold the call is refused before anything is launched
        g2 = GpuSide(par, plan)
        try:
            g2.load_keys(keys)
            if fold_steps and not set(fold_steps) <= set(ckks.required_rotations(plan)):
                with pytest.raises(g2.bf.BifrostError) as ei:
                    g2.bf.bf_fold(g2.ctx, out, n_out)
                assert ei.value.code == g2.bf.BF_ERR_MISSING_KEY
        finally:
            g2.close()
    finally:
        g.close()


def test_fold_of_more_ciphertexts_than_one_key_switch_batch():
    # 70 ciphertexts: the rounds run in two batches (64 + 6); sampled ones are compared with the oracle
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4)
    s = ckks.keygen(par, 43)
    fold_steps = ckks.fold_rotations(plan)
    keys = ckks.make_rotation_keys(par, s, plan, 43, extra_steps=fold_steps)
    n_ct = 70
    # [r][2][N] uniform residues per ciphertext, rearranged to the boundary layout [2][r][N]
    cts = np.stack([np.ascontiguousarray(wl.gen_uniform_residues(43, f"fold{t}", par.primes, (2, par.N)).transpose(1, 0, 2))
                    for t in range(n_ct)])
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys, extra_steps=fold_steps)
        d = g.to_dev(cts)
        g.bf.bf_fold(g.ctx, d, n_ct)
        got = g.to_host_u64(d)
        for t in (0, 1, 63, 64, 69):
            assert np.array_equal(got[t], ckks.fold_in_ciphertext(par, plan, cts[t], keys)), t
    finally:
        g.close()


@pytest.mark.parametrize("modes", [{}, BEST], ids=["plain", "best"])
def test_fallback_path_in_several_rounds_of_its_scratch(modes):
    # the on-the-fly path encodes output groups in rounds bounded by a scratch size: one group per round,
    # two per round with a ragged last round, and everything in one round must give the oracle's residues
    # (headline plan: rounds that start in the middle of a giant step, whose rotated parts are stored permuted)
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4, **modes)
    d_out, d_in = 150, 130                        # 3 output blocks x 4 giant steps = 12 groups of 3 x 4 terms
    s = ckks.keygen(par, 31)
    keys = ckks.make_rotation_keys(par, s, plan, 31)
    W = wl.gen_weights(31, "rounds", d_out, d_in)
    x = wl.gen_activation(31, "rounds", d_in)
    cts = ckks.encrypt_vector(par, plan, s, x, 31)
    expect = ckks.linear(par, plan, cts, W, keys)
    group_bytes = 3 * 4 * (par.r + (1 if modes else 0)) * par.N * 8
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        for bound in (1, 5 * group_bytes + 17, 2 * group_bytes, 3 * group_bytes, 1 << 32):
            g.bf.bf_set_encode_scratch(g.ctx, bound)
            got = g.to_host_u64(g.linear(cts, W, d_out, d_in))
            for p in range(plan.n_out(d_out)):
                assert np.array_equal(got[p], expect[p]), (bound, p)
        with pytest.raises(g.bf.BifrostError):
            g.bf.bf_set_encode_scratch(g.ctx, 0)
    finally:
        g.close()


def test_stacking_projections_that_share_an_input_changes_no_residue():
    # q/k/v (or gate/up) read the same activation: one call over the row-stacked matrix must give
    # exactly the ciphertexts of the separate calls
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4)
    s = ckks.keygen(par, 21)
    keys = ckks.make_rotation_keys(par, s, plan, 21)
    x = wl.gen_activation(21, "shared", 100)
    cts = ckks.encrypt_vector(par, plan, s, x, 21)
    W1 = wl.gen_weights(21, "w1", 128, 100)
    W2 = wl.gen_weights(21, "w2", 64, 100)
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        o1 = g.to_host_u64(g.linear(cts, W1, 128, 100))
        o2 = g.to_host_u64(g.linear(cts, W2, 64, 100))
        both = g.to_host_u64(g.linear(cts, np.concatenate([W1, W2]), 192, 100))
        assert np.array_equal(both[:2], o1) and np.array_equal(both[2:], o2)
        expect = ckks.linear(par, plan, cts, W2, keys)
        assert np.array_equal(o2[0], expect[0])
    finally:
        g.close()


def test_structured_matrices_on_device():
    par = oracle_params("n12")
    plan = ckks.Plan(64, 4, 4, 4)
    s = ckks.keygen(par, 5)
    keys = ckks.make_rotation_keys(par, s, plan, 5)
    x = wl.gen_activation(5, "struct", 64)
    cts = ckks.encrypt_vector(par, plan, s, x, 5)
    g = GpuSide(par, plan)
    try:
        g.load_keys(keys)
        mats = {"zero": np.zeros((64, 64), np.float32), "identity": np.eye(64, dtype=np.float32),
                "shift": np.roll(np.eye(64, dtype=np.float32), 5, axis=1)}
        single = np.zeros((64, 64), np.float32)
        single[17, 42] = 1.5
        mats["single"] = single
        for name, W in mats.items():
            got = g.to_host_u64(g.linear(cts, W, 64, 64))
            low = ckks.rescale(par, got[0])
            scale = par.scale * par.scale / par.primes[-1]
            y = ckks.fold_output(ckks.decode(ckks.decrypt(par, s, low), par.N, scale), plan, 0, 64)
            assert np.abs(y - W.astype(np.float64) @ x).max() < 1e-6, name
    finally:
        g.close()


def test_error_paths_do_not_touch_the_device():
    import torch
    from paper_2606_17421_b200 import bifrost as bf
    ps = wl.PARAM_SETS["n12"]
    plan = bf.bf_plan(64, 1, 8, 8)
    basis = list(ps["primes"]) + [ps["special"]]
    with pytest.raises(bf.BifrostError) as ei:
        bf.bf_ctx_create(ps["N"], basis[:-1] + [basis[0]], 3, 2.0 ** 40, plan)      # duplicate prime
    assert ei.value.code == bf.BF_ERR_BAD_PRIME
    with pytest.raises(bf.BifrostError) as ei:
        bf.bf_ctx_create(ps["N"], [basis[0] + 2] + basis[1:], 3, 2.0 ** 40, plan)   # not 1 mod 2N
    assert ei.value.code == bf.BF_ERR_BAD_PRIME
    with pytest.raises(bf.BifrostError) as ei:
        bf.bf_ctx_create(ps["N"], basis, 3, 2.0 ** 40, bf.bf_plan(64, 1, 8, 4))
    assert ei.value.code == bf.BF_ERR_SHAPE
    with pytest.raises(bf.BifrostError) as ei:
        bf.bf_ctx_create(3000, basis, 3, 2.0 ** 40, plan)
    assert ei.value.code == bf.BF_ERR_INVALID_ARG
    ctx = bf.bf_ctx_create(ps["N"], basis, 3, 2.0 ** 40, plan)
    try:
        ct = torch.zeros((1, 2, 3, ps["N"]), dtype=torch.int64, device="cuda")
        W = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
        with pytest.raises(bf.BifrostError) as ei:          # no keys loaded
            bf.bf_linear(ctx, ct, 1, None, W, 64, 64, ct.clone(), 1)
        assert ei.value.code == bf.BF_ERR_MISSING_KEY
        with pytest.raises(bf.BifrostError) as ei:          # wrong number of input ciphertexts
            bf.bf_linear(ctx, ct, 2, None, W, 64, 64, ct.clone(), 1)
        assert ei.value.code == bf.BF_ERR_SHAPE
        low = torch.zeros((1, 2, 2, ps["N"]), dtype=torch.int64, device="cuda")
        with pytest.raises(bf.BifrostError) as ei:          # the fused call reports the same errors
            bf.bf_linear_rescaled(ctx, ct, 1, None, W, 64, 64, low, 1)
        assert ei.value.code == bf.BF_ERR_MISSING_KEY
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_linear_rescaled(ctx, ct, 2, None, W, 64, 64, low, 1)
        assert ei.value.code == bf.BF_ERR_SHAPE
        with pytest.raises(bf.BifrostError) as ei:          # no output buffer
            bf.bf_linear_rescaled(ctx, ct, 1, None, W, 64, 64, None, 1)
        assert ei.value.code == bf.BF_ERR_INVALID_ARG
        bf.bf_set_cache_budget(ctx, 1000)
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_encode_weights(ctx, W, 64, 64)
        assert ei.value.code == bf.BF_ERR_OOM
        with pytest.raises(bf.BifrostError) as ei:          # (the budget is checked after the split)
            bf.bf_encode_weights_split(ctx, W, 64, 64, 16, 4)
        assert ei.value.code == bf.BF_ERR_OOM
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_encode_weights_split(ctx, W, 64, 64, 16, 8)
        assert ei.value.code == bf.BF_ERR_SHAPE
    finally:
        bf.bf_ctx_destroy(ctx)
