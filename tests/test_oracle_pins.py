"""Pins for the CPU oracle: each part is checked against something other than itself --
values the THC paper prints, closed forms, library routines, brute force on tiny inputs --
chosen so that a dropped term, a wrong sign or index, or a transposed operand fails."""
import ctypes
import os
from fractions import Fraction
from math import comb

import numpy as np
import pytest
from scipy.linalg import hadamard
from scipy.stats import norm

from oracle import oracle as O

SEED = 0x0123456789ABCDEF
T4_30 = (0, 3, 5, 7, 9, 11, 13, 14, 15, 17, 19, 21, 23, 25, 27, 30)
TP32 = 2.1538746940614564


def cfg(bits=4, g=30, table=T4_30, k=10, t_p=TP32, seed=SEED):
    return O.Config(bits=bits, granularity=g, table=tuple(table), t_p=t_p, log2_block=k, seed=seed)


def frac(s):
    return float(Fraction(s))


# ------------------------------------------------------------------------------- Philox
def _curand_host(seed, count, offset=0):
    path = "/usr/local/cuda/lib64/libcurand.so"
    if not os.path.exists(path):
        pytest.skip("libcurand not present")
    lib = ctypes.CDLL(path)
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:   # PHILOX4_32_10
        pytest.skip("cuRAND host generator unavailable")
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = np.zeros(count, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(count)) == 0
    lib.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 1, SEED, 0xFFFFFFFFFFFFFFFF])
@pytest.mark.parametrize("offset", [0, 4 * 65536 * 5 + 4 * 65530, (1 << 50) * 3 + 4 * 65536 * 7 + 36])
def test_philox_matches_curand_host_generator(seed, offset):
    """cuRAND's host Philox4_32_10 generator is an independent implementation of the same
    generator: its q-th group of four outputs (q = offset/4 + i) is the block with
    key = (seed lo, seed hi) and counter = (q>>16 lo, q>>16 hi, q & 0xFFFF, 0).  This pins
    the round function, the key schedule, key words and counter words 0-2."""
    groups = 24
    ref = _curand_host(seed, 4 * groups, offset)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    mine = []
    for i in range(groups):
        q = offset // 4 + i
        hi = q >> 16
        mine.append(O.philox4x32_10([hi & 0xFFFFFFFF, hi >> 32, q & 0xFFFF, 0], key))
    assert np.array_equal(ref, np.concatenate(mine))


def test_philox_every_counter_and_key_word_matters():
    base = O.philox4x32_10([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        assert not np.array_equal(base, O.philox4x32_10(c, [5, 6]))
    assert not np.array_equal(base, O.philox4x32_10([1, 2, 3, 4], [4, 6]))
    assert not np.array_equal(base, O.philox4x32_10([1, 2, 3, 4], [5, 7]))


def test_sign_and_u16_field_layout():
    """Sign bit j mod 128 of the call (j/128, ., 0xFFFFFFFF, round); 16-bit field j mod 8
    of the call (j/8, ., worker, round)."""
    key = [SEED & 0xFFFFFFFF, SEED >> 32]
    for j in [0, 1, 31, 32, 127, 128, 1000, (1 << 33) + 77]:
        call = j >> 7
        out = O.philox4x32_10([call & 0xFFFFFFFF, call >> 32, 0xFFFFFFFF, 3], key)
        bit = (int(out[(j & 127) >> 5]) >> (j & 31)) & 1
        assert O.sign(SEED, 3, j) == (-1 if bit else 1)
    for j in [0, 1, 6, 7, 8, 12345, (1 << 35) + 5]:
        call = j >> 3
        out = O.philox4x32_10([call & 0xFFFFFFFF, call >> 32, 9, 2], key)
        word = int(out[(j & 7) >> 1])
        field = (word >> 16) if (j & 1) else (word & 0xFFFF)
        assert O.u16(SEED, 2, 9, j) == field


def test_signs_balanced_and_u16_uniform():
    s = O.signs(SEED, 0, 0, 1 << 14)
    assert abs(int(s.sum())) < 4 * np.sqrt(s.size)
    assert set(np.unique(s)) == {-1, 1}
    u = np.array([O.u16(SEED, 0, 1, j) for j in range(1 << 14)])
    hist = np.bincount(u >> 12, minlength=16)
    expect = u.size / 16
    chi2 = ((hist - expect) ** 2 / expect).sum()
    assert chi2 < 45.0                       # 15 dof, p ~ 1e-4
    # different workers and rounds are different streams
    u2 = np.array([O.u16(SEED, 0, 2, j) for j in range(256)])
    u3 = np.array([O.u16(SEED, 1, 1, j) for j in range(256)])
    assert (u[:256] != u2).mean() > 0.9 and (u[:256] != u3).mean() > 0.9


# --------------------------------------------------------------------------- Hadamard
@pytest.mark.parametrize("k", [1, 2, 3, 5, 8])
def test_fwht_equals_dense_sylvester_matrix(k):
    """Small integers: every fp32 sum is exact, so the butterfly result must equal the
    dense product with scipy's Sylvester Hadamard matrix exactly."""
    B = 1 << k
    rng = np.random.default_rng(k)
    v = rng.integers(-50, 50, size=B).astype(np.float32)
    assert np.array_equal(O.fwht(v), (hadamard(B).astype(np.int64) @ v.astype(np.int64)).astype(np.float32))


def test_fwht_twice_is_B_times_identity():
    for k in (3, 6, 10):
        B = 1 << k
        v = np.random.default_rng(1).integers(-8, 8, size=B).astype(np.float32)
        assert np.array_equal(O.fwht(O.fwht(v)), B * v)


def test_hadamard_entry_is_parity_of_and():
    B = 16
    for j in range(B):
        e = np.zeros(B, dtype=np.float32)
        e[j] = 1
        col = O.fwht(e)
        expect = np.array([(-1) ** bin(i & j).count("1") for i in range(B)], dtype=np.float32)
        assert np.array_equal(col, expect)


def test_rht_brute_force_d8():
    """d = B = 8: RHT(x) = H D x / sqrt(8) and RHT^-1(v) = D H v / sqrt(8) with the dense
    matrices in float64."""
    c = cfg(k=3)
    rng = np.random.default_rng(8)
    x = rng.standard_normal(8).astype(np.float32)
    s = O.signs(SEED, 5, 0, 8).astype(np.float64)
    H = hadamard(8).astype(np.float64)
    expect = H @ (s * x.astype(np.float64)) / np.sqrt(8.0)
    got = O.rht_forward(x, c, 5)
    assert np.allclose(got, expect, rtol=0, atol=2e-6 * np.abs(expect).max())
    v = rng.standard_normal(8).astype(np.float32)
    expect_inv = s * (H @ v.astype(np.float64)) / np.sqrt(8.0)
    got_inv = O.rht_inverse(v, 8, c, 5)
    assert np.allclose(got_inv, expect_inv, rtol=0, atol=2e-6 * np.abs(expect_inv).max())
    # the two differ unless D is trivial: guards against applying D on the wrong side
    assert not np.allclose(O.rht_forward(v, c, 5), got_inv, atol=1e-3)


@pytest.mark.parametrize("k,d", [(4, 16), (6, 200), (10, 3000)])
def test_rht_preserves_norm_inverts_and_is_linear(k, d):
    c = cfg(k=k)
    rng = np.random.default_rng(d)
    x = rng.standard_normal(d).astype(np.float32)
    y = rng.standard_normal(d).astype(np.float32)
    rx = O.rht_forward(x, c, 1)
    assert rx.size == c.d_pad(d)
    assert abs(np.linalg.norm(rx.astype(np.float64)) / np.linalg.norm(x.astype(np.float64)) - 1) < 1e-6
    back = O.rht_inverse(rx, d, c, 1)
    assert np.abs(back - x).max() <= 2e-6 * np.abs(x).max() * np.sqrt(k)
    rs = O.rht_forward(x + y, c, 1)
    assert np.allclose(rs, rx + O.rht_forward(y, c, 1), atol=1e-5)
    # a different round draws a different D
    assert not np.allclose(O.rht_forward(x, c, 2), rx, atol=1e-3)


def test_rht_blocks_are_independent_and_padded_with_zeros():
    c = cfg(k=4)
    x = np.arange(1, 41, dtype=np.float32)          # d = 40 -> 3 blocks of 16, 8 pad
    r = O.rht_forward(x, c, 0)
    assert r.size == 48
    xp = np.zeros(48, dtype=np.float32)
    xp[:40] = x
    for blk in range(3):
        s = O.signs(SEED, 0, 16 * blk, 16).astype(np.float64)
        expect = hadamard(16) @ (s * xp[16 * blk:16 * blk + 16]) / 4.0
        assert np.allclose(r[16 * blk:16 * blk + 16], expect, atol=1e-5)


# ------------------------------------------------------------------------------ scales
def test_scale_closed_form_and_max_over_workers():
    c = cfg(k=5)
    rng = np.random.default_rng(3)
    x = rng.standard_normal((3, 70)).astype(np.float32)
    x[1] *= 4.0
    M = O.scales(x, c)
    assert M.size == 3
    for blk in range(3):
        seg = x[:, 32 * blk:32 * blk + 32].astype(np.float64)
        ell = np.sqrt((seg ** 2).sum(axis=1)).max()
        assert M[blk] == np.float32(TP32 * ell / np.sqrt(32.0))
    # the norm, not its square: doubling the input doubles M
    assert np.allclose(O.scales(2 * x, c), 2 * M, rtol=1e-6)


def test_t_p_is_the_normal_quantile():
    assert abs(norm.ppf(1 - (1 / 32) / 2) - TP32) < 1e-12


def test_about_p_of_the_coordinates_are_clamped():
    """Section 5.1: roughly a p fraction of the transformed coordinates falls outside
    [-M, M] when M = t_p * ||x|| / sqrt(d)."""
    k = 14
    c = cfg(k=k)
    x = np.random.default_rng(11).standard_normal((1, 1 << k)).astype(np.float32)
    M = O.scales(x, c)[0]
    r = O.rht_forward(x[0], c, 0)
    p_hat = (np.abs(r) > M).mean()
    p = 1 / 32
    se = np.sqrt(p * (1 - p) / r.size)
    assert abs(p_hat - p) < 5 * se


# ---------------------------------------------------------- quantisation: paper examples
def test_paper_tables_T0_T1_T2(golden):
    t0 = [frac(v) for v in golden["T0_values"].split()]
    t1 = [frac(v) for v in golden["T1_values"].split()]
    # T0: index sum determines value sum; T1: it does not.
    assert abs(t0[0] + t0[3]) < 1e-15 and abs(t0[1] + t0[2]) < 1e-15
    assert frac(golden["T0_index_sum_3_value_sum"]) == 0
    assert abs(t1[1] + t1[3] - frac(golden["T1_case_1_3"])) < 1e-15
    assert abs(t1[2] + t1[2] - frac(golden["T1_case_2_2"])) < 1e-15
    # T2 through the oracle: value of an index on [-1, 1]
    T2 = tuple(int(v) for v in golden["T2_table"].split())
    g = int(golden["T2_granularity"])
    c = cfg(bits=2, g=g, table=T2, k=3)
    scl = np.ones(1, dtype=np.float32)                       # M = 1, m = -1
    vals = O.dequantize(np.array([0, 1, 2, 3, 0, 0, 0, 0], dtype=np.uint8), scl, c)
    assert vals[1] == frac(golden["T2_value_of_1"]) and vals[2] == frac(golden["T2_value_of_3"])
    assert vals[0] == -1.0 and vals[3] == 1.0
    # uniform THC is the identity table with g = 2^b - 1: values are T0
    cu = cfg(bits=2, g=3, table=(0, 1, 2, 3), k=3)
    vu = O.dequantize(np.array([0, 1, 2, 3, 0, 0, 0, 0], dtype=np.uint8), scl, cu)
    assert np.allclose(vu[:4], t0, atol=1e-15)


def test_paper_three_sender_example(golden):
    """Indices (1,1,1) and (0,0,2) under T2: same table-value sum, same decoded average
    -1/2, although the index sums differ."""
    T2 = tuple(int(v) for v in golden["T2_table"].split())
    c = cfg(bits=2, g=4, table=T2, k=3)
    scl = np.ones(1, dtype=np.float32)
    a = [int(v) for v in golden["T2_three_senders_a"].split()]
    b = [int(v) for v in golden["T2_three_senders_b"].split()]
    sums = []
    for case in (a, b):
        packed = np.stack([O.pack(np.full(8, z, dtype=np.uint8), 2) for z in case])
        total = O.aggregate(packed, 8, c, 8)
        assert np.all(total == int(golden["T2_three_senders_value_sum"]))
        est = O.estimate(total, 3, scl, c)
        assert np.all(est == np.float32(-0.5))
        sums.append(total)
    assert sum(a) != sum(b)
    assert np.array_equal(sums[0], sums[1])


def test_prototype_sizing(golden):
    g = int(golden["prototype_granularity"])
    n = int(golden["prototype_max_workers"])
    assert O.acc_bits(n, g) == int(golden["prototype_sum_bits"])
    assert O.acc_bits(n + 1, g) == 16                 # 9 * 30 = 270 overflows 8 bits
    d_pad = 1 << 10
    c = cfg(k=10)
    z = np.zeros(d_pad, dtype=np.uint8)
    assert 4 * d_pad // O.pack(z, 4).size == int(golden["reduction_up"])
    total = O.aggregate(O.pack(z, 4)[None, :], d_pad, c, 8)
    assert 4 * d_pad // total.nbytes == int(golden["reduction_down"])


def test_appendixB_counts(golden):
    n, k = (int(v) for v in golden["appendixB_b4_g51_options_binomial"].split())
    assert 4.7e11 < comb(n, k) < 4.9e11
    assert comb(23, 6) == int(golden["appendixB_b4_g51_symmetric_options"])


# ------------------------------------------------- quantisation: statistical behaviour
def _p_up_reference(a, M, g, table):
    """Float64 statement of Section 4.1: interval [q0, q1] of the sub-grid containing a and
    the probability of rounding up."""
    y = (np.clip(a, -M, M) + M) * g / (2 * M)
    t = np.asarray(table, dtype=np.float64)
    z0 = np.clip(np.searchsorted(t, y, side="right") - 1, 0, len(table) - 2)
    return z0, (y - t[z0]) / (t[z0 + 1] - t[z0])


@pytest.mark.parametrize("bits,g,table", [(4, 30, T4_30), (2, 4, (0, 1, 3, 4)), (1, 1, (0, 1)),
                                          (2, 3, (0, 1, 2, 3))])
def test_quantizer_picks_the_two_neighbours_with_the_right_probability(bits, g, table):
    """For each coordinate the index is z0 or z0+1 (the neighbours on the sub-grid) and,
    over many rounds, the up-frequency matches (a - q0)/(q1 - q0) -- Section 4.1, not the
    reversed form of the appendix."""
    k = 6
    c = cfg(bits=bits, g=g, table=table, k=k)
    rng = np.random.default_rng(5)
    M = np.float32(0.75)
    r = rng.uniform(-0.9, 0.9, size=1 << k).astype(np.float32)      # some get clamped
    scl = np.full(1, M, dtype=np.float32)
    z0, p_up = _p_up_reference(r.astype(np.float64), float(M), g, table)
    rounds = 4000
    ups = np.zeros(r.size)
    for rnd in range(rounds):
        z = O.quantize(r, scl, c, rnd, worker=3)
        assert np.all((z == z0) | (z == z0 + 1))
        ups += (z == z0 + 1)
    se = np.sqrt(np.maximum(p_up * (1 - p_up), 1e-4) / rounds)
    assert np.all(np.abs(ups / rounds - p_up) < 5 * se + 1e-3)
    # pooled: catches a small systematic bias
    assert abs((ups / rounds - p_up).mean()) < 4 * np.sqrt(0.25 / (rounds * r.size))


def test_quantizer_is_unbiased_over_1e4_seeds():
    """Mean over 10^4 independent draws of the dequantised value equals clamp(r)
    (unbiasedness, Section 4.1), within 4 standard errors per coordinate and pooled; the
    per-coordinate variance is (a - q0)(q1 - a) (the integrand of Appendix B)."""
    k = 5
    c = cfg(k=k)
    M = np.float32(1.5)
    scl = np.full(1, M, dtype=np.float32)
    r = np.linspace(-1.7, 1.7, 1 << k).astype(np.float32)
    target = np.clip(r.astype(np.float64), -1.5, 1.5)
    draws = 10_000
    acc = np.zeros(r.size)
    acc2 = np.zeros(r.size)
    for s in range(draws):
        cs = cfg(k=k, seed=0x9E3779B97F4A7C15 * (s + 1) % (1 << 64))
        v = O.dequantize(O.quantize(r, scl, cs, 0, worker=0), scl, cs)
        acc += v
        acc2 += v * v
    mean = acc / draws
    var = acc2 / draws - mean ** 2
    step = 2 * 1.5 / 30
    t = np.asarray(T4_30) * step - 1.5
    z0 = np.clip(np.searchsorted(t, target, side="right") - 1, 0, 14)
    var_ref = (target - t[z0]) * (t[z0 + 1] - target)
    se = np.sqrt(var_ref / draws) + 1e-9
    assert np.all(np.abs(mean - target) < 4.5 * se + 3e-5)
    assert abs((mean - target).mean()) < 4 * np.sqrt(var_ref.mean() / (draws * r.size)) + 1e-5
    assert np.allclose(var, var_ref, rtol=0.12, atol=2e-4)


def test_identity_table_is_textbook_uniform_sq():
    """g = 2^b - 1 with the identity table: index = floor(y) + [u < frac(y)] (uniform THC,
    Section 4.2), with u the 16-bit variate; checked away from 2^-16 rounding ties."""
    k = 8
    c = cfg(bits=4, g=15, table=tuple(range(16)), k=k)
    M = np.float32(2.0)
    scl = np.full(1, M, dtype=np.float32)
    rng = np.random.default_rng(2)
    r = rng.uniform(-2.2, 2.2, size=1 << k).astype(np.float32)
    z = O.quantize(r, scl, c, 7, worker=1)
    y = (np.clip(r.astype(np.float64), -2.0, 2.0) + 2.0) * 15 / 4.0
    fl = np.minimum(np.floor(y), 14)
    fr = y - fl
    u = np.array([O.u16(SEED, 7, 1, j) for j in range(r.size)]) / 65536.0
    safe = np.abs(u - fr) > 1e-4
    assert safe.mean() > 0.99
    assert np.array_equal(z[safe], (fl + (u < fr))[safe].astype(np.uint8))


def test_quantizer_edges_and_degenerate_blocks():
    c = cfg(k=3)
    scl = np.array([1.0], dtype=np.float32)
    r = np.array([-5, -1, 1, 5, np.nan, 0, 0, 0], dtype=np.float32)
    for rnd in range(20):
        z = O.quantize(r, scl, c, rnd, 0)
        assert z[0] == 0 and z[1] == 0            # at or below m: index 0, never up
        assert z[2] == 15 and z[3] == 15          # at or above M: last index, always
        assert z[4] == 0                          # NaN coordinate -> 0
        assert z[5] in (7, 8)                     # y = 15 = T[8] exactly ... T[7] = 14
    # y exactly on a table value never rounds up
    z = np.array([O.quantize(r, scl, c, rnd, 0)[5] for rnd in range(200)])
    assert np.all(z == 8)
    # zero or non-finite scale: all indices 0, decompress gives exact zeros
    for bad in (0.0, np.inf, np.nan):
        scl_bad = np.array([bad], dtype=np.float32)
        assert np.all(O.quantize(r, scl_bad, c, 0, 0) == 0)
        out = O.decompress(np.full(8, 77, dtype=np.uint8), 4, 8, scl_bad, c, 0)
        assert np.all(out == 0.0)


# ------------------------------------------------------------------- pack / aggregate
@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_pack_layout_brute_force(bits):
    """Index j sits at bits [j*b, j*b+b) of the little-endian bit stream: for b dividing 8 at
    bit offset (j mod 8/b)*b of byte j*b/8; three-bit indices straddle bytes."""
    per = 8 // bits
    d_pad = 64
    rng = np.random.default_rng(bits)
    z = rng.integers(0, 1 << bits, size=d_pad).astype(np.uint8)
    packed = O.pack(z, bits)
    assert packed.size == d_pad * bits // 8
    bitstream = np.unpackbits(packed, bitorder="little")
    for j in range(d_pad):
        val = sum(int(bitstream[j * bits + t]) << t for t in range(bits))
        assert val == z[j]
        if 8 % bits == 0:
            assert (int(packed[j // per]) >> ((j % per) * bits)) & ((1 << bits) - 1) == z[j]
    if bits == 3:                                        # eight indices are one 24-bit integer
        for u in range(d_pad // 8):
            word = int(packed[3 * u]) | int(packed[3 * u + 1]) << 8 | int(packed[3 * u + 2]) << 16
            assert word == sum(int(z[8 * u + e]) << (3 * e) for e in range(8))
    assert np.array_equal(O.unpack(packed, d_pad, bits), z)


def test_pack_every_value_in_every_slot():
    for bits in (1, 2, 4):
        per = 8 // bits
        for slot in range(per):
            for val in range(1 << bits):
                z = np.zeros(per, dtype=np.uint8)
                z[slot] = val
                assert O.pack(z, bits)[0] == val << (slot * bits)


@pytest.mark.parametrize("bits,g,table,n,w", [(4, 30, T4_30, 8, 8), (2, 4, (0, 1, 3, 4), 5, 8),
                                              (4, 30, T4_30, 16, 16), (8, 255, tuple(range(256)), 3, 16),
                                              (1, 1, (0, 1), 32, 8), (8, 255, tuple(range(256)), 300, 32)])
def test_aggregate_is_the_sum_of_table_values(bits, g, table, n, w):
    c = cfg(bits=bits, g=g, table=table, k=6)
    d_pad = 128
    rng = np.random.default_rng(n)
    z = rng.integers(0, 1 << bits, size=(n, d_pad)).astype(np.uint8)
    z[:, 0] = (1 << bits) - 1                      # the maximum n*g must survive
    packed = np.stack([O.pack(z[i], bits) for i in range(n)])
    total = O.aggregate(packed, d_pad, c, w)
    expect = np.asarray(table, dtype=np.int64)[z].sum(axis=0)
    assert expect[0] == n * g
    assert total.dtype.itemsize * 8 == w
    assert np.array_equal(total.astype(np.int64), expect)
    # little-endian storage of the sums
    raw = total.view(np.uint8).reshape(d_pad, w // 8)
    assert np.array_equal(sum(raw[:, t].astype(np.int64) << (8 * t) for t in range(w // 8)), expect)


# ----------------------------------------------------------- decompress / homomorphism
def test_estimate_closed_form_and_single_worker_case():
    c = cfg(k=4)
    scl = np.array([0.5, 2.0], dtype=np.float32)
    total = np.arange(32, dtype=np.uint8) * 3
    est = O.estimate(total, 4, scl, c)
    M = np.repeat(scl.astype(np.float64), 16)
    expect = -M + total / 4.0 * (2 * M / 30.0)
    assert np.allclose(est, expect, rtol=0, atol=2e-7 * M)
    # n = 1: the estimate of a single worker's table values is its dequantised vector
    z = (np.arange(32) % 16).astype(np.uint8)
    one = O.aggregate(O.pack(z, 4)[None, :], 32, c, 8)
    assert np.allclose(O.estimate(one, 1, scl, c), O.dequantize(z, scl, c), atol=2e-7 * M.max())


def test_homomorphic_identity():
    """Definition 3: decompressing the integer sum equals the average of the per-worker
    dequantised vectors -- before and after the (linear) inverse RHT."""
    k, n, d = 7, 6, 300
    c = cfg(k=k)
    x = np.random.default_rng(4).standard_normal((n, d)).astype(np.float32)
    res = O.thc_round(x, c, rnd=2)
    scl = res["scales"]
    d_pad = c.d_pad(d)
    zs = [O.unpack(res["packed"][i], d_pad, 4) for i in range(n)]
    # exact in integers
    assert np.array_equal(res["sum"].astype(np.int64),
                          sum(np.asarray(T4_30, dtype=np.int64)[z] for z in zs))
    mean_deq = np.mean([O.dequantize(z, scl, c) for z in zs], axis=0)
    est = O.estimate(res["sum"], n, scl, c)
    Mmax = float(scl.max())
    assert np.abs(est - mean_deq).max() <= 4e-7 * Mmax
    out_ref = O.rht_inverse(mean_deq.astype(np.float32), d, c, 2)
    assert np.abs(res["out"] - out_ref).max() <= 1e-5 * Mmax


def test_whole_round_error_falls_with_workers_and_bits():
    """Independent unbiased rounding: NMSE of the average ~ 1/n (Appendix A.2), and 4 bits
    beat 2 bits by a wide margin (Appendix D.4: roughly an order of magnitude per extra bit)."""
    k, d = 10, 4096
    rng = np.random.default_rng(9)
    base = rng.standard_normal(d).astype(np.float32)

    def nmse(n, c):
        x = np.tile(base, (n, 1))
        out = O.thc_round(x, c, rnd=0)["out"]
        clamp_free = base.astype(np.float64)
        return float(((out - clamp_free) ** 2).sum() / (clamp_free ** 2).sum())

    # a wide range (p tiny) so that truncation bias does not mask the 1/n law
    wide = dict(t_p=4.5)
    e1 = nmse(1, cfg(k=k, **wide))
    e16 = nmse(16, cfg(k=k, **wide))
    assert 8 < e1 / e16 < 32
    e_b2 = nmse(4, cfg(bits=2, g=3, table=(0, 1, 2, 3), k=k, **wide))
    e_b4 = nmse(4, cfg(k=k, **wide))
    assert e_b2 / e_b4 > 20


def test_round_output_close_to_true_mean():
    k, n, d = 12, 8, 10_000
    c = cfg(k=k)
    x = np.random.default_rng(21).standard_normal((n, d)).astype(np.float32)
    out = O.thc_round(x, c)["out"]
    mean = x.astype(np.float64).mean(axis=0)
    nm = ((out - mean) ** 2).sum() / (mean ** 2).sum()
    assert nm < 0.2
    assert abs(np.corrcoef(out, mean)[0, 1]) > 0.9


def test_bf16_upcast_is_exact():
    bits = np.array([0x3F80, 0xBF80, 0x0001, 0x7F7F, 0x8000], dtype=np.uint16)
    f = O.bf16_to_f32(bits)
    assert f[0] == 1.0 and f[1] == -1.0 and f[4] == 0.0 and np.signbit(f[4])
    assert f[2] > 0 and f[3] == np.float32(3.3895314e38)


def test_nonfinite_norm_of_any_worker_makes_the_block_degenerate():
    c = cfg(k=4)
    x = np.ones((3, 32), dtype=np.float32)
    x[0, 3] = np.nan          # first worker: must not be overwritten by later finite norms
    x[2, 20] = np.inf         # last worker
    M = O.scales(x, c)
    assert M[0] == 0.0 and M[1] == 0.0
    x = np.ones((3, 32), dtype=np.float32)
    x[1, 16:] = 0
    assert np.all(O.scales(x, c) > 0)


def test_slice_forms_agree_with_the_whole_vector():
    """Transforming / quantising one block of a long vector with its coordinate offset gives
    the same result as processing the whole vector (blocks are independent; only the sign
    diagonal and the rounding variates depend on the global coordinate)."""
    k, d = 6, 64 * 5 - 7
    c = cfg(k=k)
    x = np.random.default_rng(17).standard_normal((2, d)).astype(np.float32)
    scl = O.scales(x, c)
    whole = O.rht_forward(x[1], c, 3)
    zw = O.quantize(whole, scl, c, 3, worker=1)
    vals = np.random.default_rng(18).standard_normal(c.d_pad(d)).astype(np.float32)
    inv_whole = O.rht_inverse(vals, d, c, 3)
    for blk in (0, 2, 4):
        lo, hi = 64 * blk, min(d, 64 * blk + 64)
        part = O.rht_forward(x[1, lo:hi], c, 3, j_base=lo)
        assert np.array_equal(part.view(np.uint32), whole[lo:lo + 64].view(np.uint32))
        zp = O.quantize(part, scl[blk:blk + 1], c, 3, worker=1, j_base=lo)
        assert np.array_equal(zp, zw[lo:lo + 64])
        ip = O.rht_inverse(vals[lo:lo + 64], hi - lo, c, 3, j_base=lo)
        assert np.array_equal(ip.view(np.uint32), inv_whole[lo:hi].view(np.uint32))


# ------------------------------------------------------------------- error feedback
def test_error_feedback_is_the_residual_of_the_workers_own_quantised_vector():
    """e = x - RHT^-1(X): equals x minus the decompression of a one-worker aggregate with
    divisor 1 (Definition 3 with n = 1), so x = e + RHT^-1(X) up to one rounding."""
    k, d = 8, 700
    c = cfg(k=k)
    x = np.random.default_rng(31).standard_normal((3, d)).astype(np.float32)
    scl = O.scales(x, c)
    for i in range(3):
        z = O.quantize(O.rht_forward(x[i], c, 4), scl, c, 4, i)
        e = O.error_feedback(x[i], z, scl, c, 4)
        one = O.aggregate(O.pack(z, 4)[None, :], c.d_pad(d), c, 8)
        back = O.decompress(one, 1, d, scl, c, 4)
        assert np.array_equal(e, x[i] - back)
        # the residual is small: 4-bit THC keeps a few per cent NMSE per worker
        assert (e.astype(np.float64) ** 2).sum() < 0.1 * (x[i].astype(np.float64) ** 2).sum()


def test_error_feedback_removes_the_truncation_bias_over_rounds():
    """Section 5.1: truncation makes THC biased; with error feedback the running average of
    the decompressed vectors converges to the true vector, because
    sum_r RHT^-1(X^r) = R x - e^R and e stays bounded.  Without feedback the bias stays."""
    k, d, R = 8, 256, 60
    c = cfg(k=k, t_p=0.8)                      # aggressive truncation: about 42 % clamped
    rng = np.random.default_rng(33)
    grad = rng.standard_normal(d).astype(np.float32)
    e = np.zeros(d, dtype=np.float32)
    acc_ef = np.zeros(d)
    acc_plain = np.zeros(d)
    for r in range(R):
        x = (grad + e).astype(np.float32)
        scl = O.scales(x[None, :], c)
        z = O.quantize(O.rht_forward(x, c, r), scl, c, r, 0)
        one = O.aggregate(O.pack(z, 4)[None, :], d, c, 8)
        acc_ef += O.decompress(one, 1, d, scl, c, r)
        e = O.error_feedback(x, z, scl, c, r)
        scl0 = O.scales(grad[None, :], c)
        z0 = O.quantize(O.rht_forward(grad, c, r), scl0, c, r, 0)
        acc_plain += O.decompress(O.aggregate(O.pack(z0, 4)[None, :], d, c, 8), 1, d, scl0, c, r)
    g64 = grad.astype(np.float64)
    err_ef = np.linalg.norm(acc_ef / R - g64) / np.linalg.norm(g64)
    err_plain = np.linalg.norm(acc_plain / R - g64) / np.linalg.norm(g64)
    assert err_ef < 0.05
    assert err_plain > 3 * err_ef
    # exactly: R * mean = R * grad - e^R (up to fp32 rounding of the additions)
    assert np.allclose(acc_ef, R * g64 - e, atol=2e-4 * R)


# ------------------------------------------------- exact range (Algorithm 1's preliminary stage)
def test_ranges_are_min_and_max_of_the_dense_rotation():
    """(lo, hi) per block = min and max over workers and coordinates of (1/sqrt B) H D x,
    written out with SciPy's dense Sylvester matrix in float64."""
    k, n, d = 4, 3, 37                                     # three blocks of 16, the last ragged
    c = cfg(k=k)
    rng = np.random.default_rng(11)
    x = rng.standard_normal((n, d)).astype(np.float32)
    lo, hi = O.ranges(x, c, 5)
    B = 1 << k
    H = hadamard(B).astype(np.float64)
    for blk in range(3):
        vals = []
        for i in range(n):
            xp = np.zeros(3 * B)
            xp[:d] = x[i]
            s = O.signs(c.seed, 5, blk * B, B).astype(np.float64)
            vals.append(H @ (s * xp[blk * B:(blk + 1) * B]) / np.sqrt(B))
        vals = np.concatenate(vals)
        assert abs(lo[blk] - vals.min()) <= 1e-6 and abs(hi[blk] - vals.max()) <= 1e-6
        assert lo[blk] < 0.0 < hi[blk]


def test_symmetric_range_is_the_special_case_lo_equals_minus_hi():
    """The general [lo, hi] quantiser and decoder with lo = -M reproduce the Section 5.3 path
    bit for bit (kappa = 1/(2M), offset = 1/2 exactly)."""
    c = cfg(k=8)
    rng = np.random.default_rng(3)
    r = rng.standard_normal(4 * 256).astype(np.float32)
    scl = np.array([0.7, 2.0, 1e-3, 3.3], np.float32)
    z0 = O.quantize(r, scl, c, rnd=2, worker=1)
    z1 = O.quantize(r, scl, c, rnd=2, worker=1, lo=-scl)
    assert np.array_equal(z0, z1)
    tot = O.aggregate(O.pack(z0, 4)[None, :], r.size, c, 8)
    assert np.array_equal(O.estimate(tot, 1, scl, c).view(np.uint32),
                          O.estimate(tot, 1, scl, c, lo=-scl).view(np.uint32))


def test_exact_range_clamps_nothing_and_decodes_without_bias():
    """With Algorithm 1's exact range no coordinate is truncated: the block's minimum gets
    index 0 and decodes to lo, its maximum gets the last index and decodes to hi, and the
    mean of the decoded value over independent rounding draws (different worker ids, same
    rotation) approaches r at every coordinate, extremes included."""
    k = 6
    c = cfg(k=k)
    rng = np.random.default_rng(19)
    x = (rng.standard_normal((1, 64)) * np.exp(rng.standard_normal((1, 64)))).astype(np.float32)
    lo, hi = O.ranges(x, c, 0)
    r = O.rht_forward(x[0], c, 0)
    assert r.min() == lo[0] and r.max() == hi[0]
    draws = 4000
    acc = np.zeros(64)
    acc2 = np.zeros(64)
    for wkr in range(draws):
        z = O.quantize(r, hi, c, rnd=0, worker=wkr, lo=lo)
        if wkr == 0:
            assert z[np.argmin(r)] == 0 and z[np.argmax(r)] == 15
        tot = O.aggregate(O.pack(z, 4)[None, :], 64, c, 8)
        v = O.estimate(tot, 1, hi, c, lo=lo).astype(np.float64)
        acc += v
        acc2 += v * v
    mean = acc / draws
    sd = np.sqrt(np.maximum(acc2 / draws - mean ** 2, 0.0) / draws)
    width = float(hi[0]) - float(lo[0])
    assert np.all(np.abs(mean - r) <= 4.5 * sd + 3e-5 * width)
    assert abs(mean[np.argmin(r)] - lo[0]) <= 1e-6 * width and abs(mean[np.argmax(r)] - hi[0]) <= 1e-6 * width


def test_uniform_thc_is_textbook_usq_on_the_exact_range():
    """Algorithm 1: identity table with g = 2^b - 1 on [m, M]: the index is floor((r-m)/(M-m) g)
    or one more, and the estimate line is m + (X/n) (M-m)/(2^b-1)."""
    b, g, k = 2, 3, 5
    c = cfg(bits=b, g=g, table=(0, 1, 2, 3), k=k)
    rng = np.random.default_rng(23)
    x = rng.standard_normal((2, 32)).astype(np.float32)
    lo, hi = O.ranges(x, c, 1)
    width = float(hi[0]) - float(lo[0])
    zs = []
    for i in range(2):
        r = O.rht_forward(x[i], c, 1)
        z = O.quantize(r, hi, c, rnd=1, worker=i, lo=lo)
        pos = (r.astype(np.float64) - float(lo[0])) / width * g
        fl = np.minimum(np.floor(pos + 1e-9), g - 1)
        assert np.all((z == fl) | (z == fl + 1) | (np.abs(pos - np.round(pos)) < 1e-5))
        zs.append(z)
    X = zs[0].astype(np.int64) + zs[1]
    tot = O.aggregate(np.stack([O.pack(z, b) for z in zs]), 32, c, 8)
    assert np.array_equal(tot.astype(np.int64), X)
    v = O.estimate(tot, 2, hi, c, lo=lo)
    expect = float(lo[0]) + X / 2.0 * width / (2 ** b - 1)
    assert np.allclose(v, expect, rtol=0, atol=2e-6 * width)


def test_exact_range_round_has_no_truncation_error_on_heavy_tails():
    """Whole rounds on heavy-tailed input with a tight clamp (p = 1/2): the norm-based range
    truncates and the error of the average stays large however many workers there are; the
    exact range only has quantisation noise, which the average over workers shrinks."""
    k, n, d = 8, 32, 512
    tight = cfg(k=k, t_p=0.6744897501960817)               # p = 1/2
    rng = np.random.default_rng(29)
    base = (rng.standard_normal(d) * np.exp(1.5 * rng.standard_normal(d))).astype(np.float32)
    x = np.tile(base, (n, 1))
    out_norm = O.thc_round(x, tight, 3)["out"].astype(np.float64)
    out_exact = O.thc_round(x, tight, 3, exact_range=True)["out"].astype(np.float64)
    e_norm = ((out_norm - base) ** 2).sum() / (base.astype(np.float64) ** 2).sum()
    e_exact = ((out_exact - base) ** 2).sum() / (base.astype(np.float64) ** 2).sum()
    assert e_exact < 0.05 and e_norm > 5 * e_exact


def test_exact_range_constant_block_decodes_to_the_constant():
    """One non-zero coordinate in the first position of a block rotates to a constant block
    (column 0 of H is all ones): min = max, every index is 0, and the estimate line
    m + X (M - m)/g with M = m returns m, so the round reproduces the input."""
    k = 4
    c = cfg(k=k)
    x = np.zeros((1, 48), np.float32)
    x[0, 16] = 3.25                                       # first coordinate of block 1
    x[0, 5] = -1.0
    lo, hi = O.ranges(x, c, 2)
    assert lo[1] == hi[1] and abs(abs(lo[1]) - 3.25 / 4.0) < 1e-7 and lo[2] == 0.0 == hi[2]
    out = O.thc_round(x, c, 2, exact_range=True)
    z = O.unpack(out["packed"][0], 48, 4)
    assert not z[16:48].any()
    assert out["out"][16] == np.float32(3.25) and not out["out"][17:].any()


# -------------------------------------- error feedback on a general (asymmetric) range [m, M]
def _dense_inverse_rht(v, d, c, rnd):
    """D (1/sqrt B) H v per block, written out with SciPy's dense Sylvester matrix in float64."""
    B = c.block
    H = hadamard(B).astype(np.float64)
    out = np.zeros(v.size)
    for blk in range(v.size // B):
        s = O.signs(c.seed, rnd, blk * B, B).astype(np.float64)
        out[blk * B:(blk + 1) * B] = s * (H @ v[blk * B:(blk + 1) * B]) / np.sqrt(B)
    return out[:d]


def test_error_feedback_on_an_asymmetric_range_follows_algorithm_2s_estimate_line():
    """Algorithm 3's e_i = x_i - RHT^-1(X_i) with Algorithm 2's quantisation values on [m, M]:
    X[j] = m + T[z[j]] (M - m)/g.  The range here is the exact, asymmetric one (m != -M) and
    differs per block.  Checked three ways: bit for bit against x minus the decompression of
    the worker's own one-worker aggregate with divisor 1 on the same range; against the
    formula written out densely in float64 (a step of 2M/g or a base of -M instead of m is
    off by a sizeable fraction of the range and fails); and by the size of the residual."""
    k, d, rnd = 6, 150, 7                                  # three blocks of 64, the last ragged
    c = cfg(k=k)
    rng = np.random.default_rng(41)
    x = (rng.standard_normal((2, d)) + 0.6 * rng.standard_normal((2, 1))).astype(np.float32)
    x[:, 70] += 9.0                                       # one-sided outlier: a lopsided range
    lo, hi = O.ranges(x, c, rnd)
    assert np.all(np.abs(lo + hi) > 0.05 * (hi - lo))      # really asymmetric, every block
    T = np.array(T4_30, np.float64)
    B = 1 << k
    for i in range(2):
        z = O.quantize(O.rht_forward(x[i], c, rnd), hi, c, rnd, i, lo=lo)
        e = O.error_feedback(x[i], z, hi, c, rnd, lo=lo)
        one = O.aggregate(O.pack(z, 4)[None, :], c.d_pad(d), c, 8)
        back = O.decompress(one, 1, d, hi, c, rnd, lo=lo)
        assert np.array_equal(e.view(np.uint32), (x[i] - back).view(np.uint32))
        m = np.repeat(lo.astype(np.float64), B)
        M = np.repeat(hi.astype(np.float64), B)
        X = m + T[z] * (M - m) / 30.0
        dense = x[i].astype(np.float64) - _dense_inverse_rht(X, d, c, rnd)
        width = float((hi - lo).max())
        assert np.abs(e - dense).max() <= 2e-6 * width
        # the two plausible slips are far outside that tolerance
        wrong_step = x[i].astype(np.float64) - _dense_inverse_rht(m + T[z] * (2.0 * M) / 30.0, d, c, rnd)
        wrong_base = x[i].astype(np.float64) - _dense_inverse_rht(-M + T[z] * (M - m) / 30.0, d, c, rnd)
        assert np.abs(e - wrong_step).max() > 1e-2 * width
        assert np.abs(e - wrong_base).max() > 1e-2 * width
        # nothing is clamped on the exact range, so the residual is quantisation noise only:
        # per rotated coordinate at most (gap/g)^2 (M-m)^2 / 4, gap <= 3 of g = 30
        nmse_bound = ((3.0 / 30.0) ** 2 / 4.0) * (width ** 2) * c.d_pad(d)
        assert (e.astype(np.float64) ** 2).sum() <= nmse_bound


def test_error_feedback_telescopes_over_rounds_on_the_exact_range():
    """Algorithm 3 with the exact range of Algorithm 1's preliminary stage: x^r = grad + e^r,
    e^{r+1} = x^r - RHT^-1(X^r), so sum_r RHT^-1(X^r) = R grad - e^R; nothing is truncated, so
    e stays at quantisation-noise size and the running mean converges to grad."""
    k, d, R = 6, 128, 40
    c = cfg(k=k)
    rng = np.random.default_rng(43)
    grad = (rng.standard_normal(d) + 0.8).astype(np.float32)   # a mean offset: m != -M in block 0
    e = np.zeros(d, np.float32)
    sent = np.zeros(d)
    for r in range(R):
        x = (grad + e).astype(np.float32)
        lo, hi = O.ranges(x[None, :], c, r)
        z = O.quantize(O.rht_forward(x, c, r), hi, c, r, 0, lo=lo)
        one = O.aggregate(O.pack(z, 4)[None, :], d, c, 8)
        sent += O.decompress(one, 1, d, hi, c, r, lo=lo)
        e = O.error_feedback(x, z, hi, c, r, lo=lo)
    g64 = grad.astype(np.float64)
    assert np.allclose(sent, R * g64 - e, atol=2e-5 * R)
    assert np.linalg.norm(e) < 0.5 * np.linalg.norm(g64)
    assert np.linalg.norm(sent / R - g64) < 0.02 * np.linalg.norm(g64)


# ------------------------------------------------ the rounding threshold, in exact arithmetic
def _rn32(q):
    """Nearest fp32 (ties to even) of a positive rational, as a Fraction (normal range)."""
    q = Fraction(q)
    e = 0
    while q / Fraction(2) ** e >= 1 << 24:
        e += 1
    while q / Fraction(2) ** e < 1 << 23:
        e -= 1
    scaled = q / Fraction(2) ** e
    m = scaled.numerator // scaled.denominator
    rem = scaled - m
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and m % 2 == 1):
        m += 1
    return Fraction(m) * Fraction(2) ** e


def test_rounding_threshold_is_the_probability_of_section_4_1_in_sixteen_bits():
    """Section 4.1: a in [q0, q1] goes up with probability (a - q0)/(q1 - q0).  For every
    coordinate the oracle rounds up exactly for the 16-bit variates below a threshold; over
    many workers (independent variates, same rotated value) the largest variate that went up
    and the smallest that did not bracket that threshold.  The bracket must contain
    RN(2^16 delta / gap) evaluated in exact rational arithmetic from the fp32 inputs
    (position u = RN(r/(2M) + 1/2), delta = RN(u g - T[z0]), R16 = RN(65536/gap))."""
    k, g = 6, 30
    c = cfg(k=k)
    rng = np.random.default_rng(47)
    r = (rng.standard_normal(64) * 0.4).astype(np.float32)
    M = np.array([1.0], np.float32)                      # kappa = 1/2, offset = 1/2: both exact
    workers = 6000
    zs = np.stack([O.quantize(r, M, c, rnd=9, worker=w) for w in range(workers)])
    us = np.array([[O.u16(c.seed, 9, w, j) for j in range(64)] for w in range(0, workers, 60)])
    T = T4_30
    checked = 0
    for j in range(64):
        u = _rn32(Fraction(float(r[j])) / 2 + Fraction(1, 2)) if r[j] > -1.0 else Fraction(0)
        u = min(max(u, Fraction(0)), Fraction(1))
        f = min(int(u * g), g - 1)
        z0 = max(z for z in range(15) if T[z] <= f)
        gap = T[z0 + 1] - T[z0]
        exact = u * g - T[z0]
        delta = _rn32(exact) if exact > 0 else Fraction(0)
        r16 = _rn32(Fraction(65536, gap))
        prod = delta * r16
        thr = prod.numerator // prod.denominator
        rem = prod - thr
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and thr % 2 == 1):
            thr += 1
        assert set(np.unique(zs[:, j])) <= {z0, z0 + 1}
        # every sampled worker's decision agrees with u16 < thr
        for row, w in enumerate(range(0, workers, 60)):
            assert (zs[w, j] == z0 + 1) == (us[row, j] < thr)
            checked += 1
        # and the up-frequency over all workers is thr / 65536 within sampling error
        freq = (zs[:, j] == z0 + 1).mean()
        p = thr / 65536.0
        assert abs(freq - p) <= 4.5 * np.sqrt(max(p * (1 - p), 1e-4) / workers)
    assert checked == 64 * 100
