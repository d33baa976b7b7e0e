"""Pins of the projection-pair oracle (u' = z + W_o a, q = W_q N_1(u')) against what the mathematics fixes:
one-hot inputs that read out single weight columns, exact row sums, power-of-two equivariance (exact in
binary floating point), a PyTorch fp64 library route, exact rational brute force on a tiny case, and the
nearest-bf16 property of every rounding.  None of them calls the oracle to check the oracle."""
import math
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import torch

from oracle import qf_oracle as orc


def bits_to_f64(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bits(x):
    """nearest binary32, then nearest bf16, ties to even (written out here, not taken from the oracle)"""
    u = np.asarray(x, np.float64).astype(np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def rand_bits(rng, shape, scale=1.0):
    return f64_to_bits(rng.standard_normal(shape) * scale)


def test_one_hot_attention_reads_out_a_column_of_w_o():
    rng = np.random.default_rng(1)
    M, d, n = 5, 24, 40                        # deliberately not square: a transposed weight fails here
    w_o, w_q, g = rand_bits(rng, (d, n)), rand_bits(rng, (n, d)), rand_bits(rng, (d,))
    a = np.zeros((M, n), np.float32)
    cols = [0, 7, 39, 13, 21]
    for m, j in enumerate(cols):
        a[m, j] = 1.0
    z = np.zeros((M, d), np.uint16)
    u, _ = orc.project_pair(a, z, w_o, g, w_q)
    for m, j in enumerate(cols):
        assert np.array_equal(u[m], w_o[:, j])            # bit for bit: 1.0 * w + 0 needs no rounding


def test_zero_w_o_passes_the_stream_through_and_unit_norm_gives_row_sums_of_w_q():
    rng = np.random.default_rng(2)
    M, d, n = 3, 64, 48
    w_o = np.zeros((d, n), np.uint16)
    w_q = rand_bits(rng, (n, d))
    a = rng.standard_normal((M, n)).astype(np.float32)
    z = rand_bits(rng, (M, d))
    g = f64_to_bits(np.ones(d))
    u, _ = orc.project_pair(a, z, w_o, g, w_q)
    assert np.array_equal(u, z)
    # a constant stream c normalises to sign(c) exactly when eps = 0, so q = +-(row sums of W_q)
    for c in (0.75, -3.0, 2.0 ** -20):
        zc = f64_to_bits(np.full((M, d), c))
        _, q = orc.project_pair(a, zc, w_o, g, w_q, eps=0.0)
        rows = np.array([math.fsum(bits_to_f64(w_q[o]).tolist()) for o in range(n)])   # exact sums
        assert np.array_equal(q[0], f64_to_bits(np.sign(c) * rows))
        assert np.array_equal(q[0], q[1]) and np.array_equal(q[0], q[2])


def test_power_of_two_scalings_are_exact():
    rng = np.random.default_rng(3)
    M, d, n = 4, 128, 96
    w_o, w_q, g = rand_bits(rng, (d, n), 0.1), rand_bits(rng, (n, d), 0.1), rand_bits(rng, (d,))
    a = rng.standard_normal((M, n)).astype(np.float32)
    z = rand_bits(rng, (M, d))
    u1, q1 = orc.project_pair(a, z, w_o, g, w_q, eps=0.0)
    # the whole stream times 4: u' shifts its exponent, N_1 (eps = 0) is scale-free, q is bit-identical
    u4, q4 = orc.project_pair(a * 4, f64_to_bits(bits_to_f64(z) * 4), w_o, g, w_q, eps=0.0)
    assert np.array_equal(bits_to_f64(u4), bits_to_f64(u1) * 4)
    assert np.array_equal(q4, q1)
    # the gain times 2: x doubles, q doubles
    _, q2 = orc.project_pair(a, z, w_o, f64_to_bits(bits_to_f64(g) * 2), w_q, eps=0.0)
    assert np.array_equal(bits_to_f64(q2), bits_to_f64(q1) * 2)
    # W_q times 1/8
    _, q8 = orc.project_pair(a, z, w_o, g, f64_to_bits(bits_to_f64(w_q) / 8), eps=0.0)
    assert np.array_equal(bits_to_f64(q8), bits_to_f64(q1) / 8)


def test_against_pytorch_fp64_and_every_rounding_is_to_nearest():
    rng = np.random.default_rng(4)
    M, d, n = 6, 256, 512
    w_o, w_q, g = rand_bits(rng, (d, n), 0.05), rand_bits(rng, (n, d), 0.05), rand_bits(rng, (d,))
    a = rng.standard_normal((M, n)).astype(np.float32)
    z = rand_bits(rng, (M, d))
    eps = 1e-6
    u, q, ue, qe = orc.project_pair(a, z, w_o, g, w_q, eps=eps, exact=True)
    t = lambda b: torch.from_numpy(bits_to_f64(b))
    a_b = t(f64_to_bits(a))
    u_t = t(z) + a_b @ t(w_o).T
    assert torch.allclose(torch.from_numpy(ue), u_t, rtol=1e-13, atol=1e-13)
    # nearest bf16 (through binary32): the oracle's bits are within half a bf16 ulp of the exact value
    uv = bits_to_f64(u)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ue), 1e-300))) - 7)
    assert (np.abs(uv - ue) <= 0.5 * ulp * (1 + 2.0 ** -14)).all()
    assert np.array_equal(u, f64_to_bits(ue))
    x_t = torch.nn.functional.rms_norm(t(u), (d,), weight=t(g), eps=eps)          # library routine, fp64
    x_b = t(f64_to_bits(x_t.numpy()))
    q_t = x_b @ t(w_q).T
    assert torch.allclose(torch.from_numpy(qe), q_t, rtol=1e-12, atol=1e-12)
    assert np.array_equal(q, f64_to_bits(qe))


def test_exact_rational_brute_force_on_a_tiny_case():
    getcontext().prec = 80
    rng = np.random.default_rng(5)
    M, d, n = 2, 4, 3
    w_o, w_q, g = rand_bits(rng, (d, n)), rand_bits(rng, (n, d)), rand_bits(rng, (d,))
    a = rng.standard_normal((M, n)).astype(np.float32)
    z = rand_bits(rng, (M, d))
    eps = 1e-5
    u, q = orc.project_pair(a, z, w_o, g, w_q, eps=eps)
    F = lambda b: Fraction(float(bits_to_f64(np.uint16(b))))
    for m in range(M):
        ab = [Fraction(float(bits_to_f64(f64_to_bits(np.float64(a[m, k]))))) for k in range(n)]
        ur = [F(z[m, o]) + sum(F(w_o[o, k]) * ab[k] for k in range(n)) for o in range(d)]
        ub = [f64_to_bits(np.float64(float(x))) for x in ur]           # float(Fraction) is correctly rounded
        assert [int(x) for x in ub] == [int(x) for x in u[m]]
        uu = [F(b) for b in ub]
        ms = sum(x * x for x in uu) / d + Fraction(eps)
        rstd = Decimal(1) / (Decimal(ms.numerator) / Decimal(ms.denominator)).sqrt()
        xs = []
        for i in range(d):
            val = Decimal(F(g[i]).numerator) / Decimal(F(g[i]).denominator) * \
                Decimal(uu[i].numerator) / Decimal(uu[i].denominator) * rstd
            xs.append(F(f64_to_bits(np.float64(float(val)))))
        for o in range(n):
            acc = sum(F(w_q[o, k]) * xs[k] for k in range(d))
            assert int(f64_to_bits(np.float64(float(acc)))) == int(q[m, o])


def test_large_eps_limit_and_zero_stream():
    rng = np.random.default_rng(6)
    M, d, n = 2, 32, 16
    w_o = np.zeros((d, n), np.uint16)
    w_q, g = rand_bits(rng, (n, d)), rand_bits(rng, (d,))
    a = np.zeros((M, n), np.float32)
    # an all-zero stream normalises to zero (no 0/0: eps > 0), so q = 0
    _, q0 = orc.project_pair(a, np.zeros((M, d), np.uint16), w_o, g, w_q, eps=1e-6)
    assert (bits_to_f64(q0) == 0).all()
    # eps far above the mean square: N_1(u) -> g u / sqrt(eps), here with sqrt(eps) = 2^10 exactly
    z = rand_bits(rng, (M, d), 2.0 ** -12)
    _, q, _, qe = orc.project_pair(a, z, w_o, g, w_q, eps=2.0 ** 20, exact=True)
    x = bits_to_f64(f64_to_bits(bits_to_f64(g) * bits_to_f64(z) / 1024.0))
    ref = x @ bits_to_f64(w_q).T
    assert np.allclose(qe, ref, rtol=1e-6, atol=0)       # mean square 2^-24 against eps 2^20: relative 2^-45
