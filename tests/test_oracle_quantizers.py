"""Pins for the oracle's quantizers, helpers and random stream.

Brute-force nearest-level search (Eq. 1, Eq. 6 with xi = 0), round-trip
invariants, the packed layout against Python's big integers, Philox against the
published known-answer vectors, and the specified log2 / exp2 against numpy.
"""
import math

import numpy as np
import pytest

import oracle

ALL_KINDS = [oracle.DE_SIGNED, oracle.DE_UNSIGNED, oracle.LINEAR_UNSIGNED, oracle.LINEAR_SIGNED,
             oracle.LINEAR_NOZERO]


def brute_nearest(levels, r):
    """argmin_k |r - y_k| by exhaustive search in binary64, first minimum wins."""
    d = np.abs(np.float64(r) - levels.astype(np.float64))
    return int(np.argmin(d)), np.sort(d)[:2]


@pytest.mark.parametrize("kind", ALL_KINDS)
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_nearest_matches_brute_force(kind, bits):
    y = oracle.codebook(kind, bits)
    rng = np.random.default_rng(bits * 10 + kind)
    lo = -1.0 if kind in (oracle.DE_SIGNED, oracle.LINEAR_SIGNED) else 0.0
    grid = np.concatenate([np.linspace(lo, 1.0, 257), rng.uniform(lo, 1.0, 600),
                           y, (y[:-1] + y[1:]) / 2, rng.normal(0, 0.01, 100).clip(lo, 1)])
    for r in grid.astype(np.float32):
        q = oracle.quant_nearest(y, float(r))
        qb, (d0, d1) = brute_nearest(y, r)
        if d1 - d0 > 1e-7:          # away from an exact tie the answer is unique
            assert q == qb, (kind, bits, r, q, qb)
        else:                       # at a tie either neighbour is nearest; the rule is "lower"
            assert abs(np.float64(r) - y[q]) <= d0 + 1e-7
    # exact midpoints that are representable go to the lower index
    y2 = oracle.codebook(oracle.LINEAR_NOZERO, 2)       # 0.25 0.5 0.75 1
    assert oracle.quant_nearest(y2, 0.375) == 0 and oracle.quant_nearest(y2, 0.625) == 1


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_log_quantizer_matches_brute_force_in_log_domain(bits):
    """Eq. 6 with xi = 0 picks the level alpha^k nearest to r in the log domain."""
    K = 1 << bits
    rng = np.random.default_rng(bits)
    for _ in range(300):
        delta = float(np.float32(math.exp(rng.uniform(-20, 3))))
        rho = math.exp(rng.uniform(math.log(1e-6), math.log(0.9)))
        alpha, inv_lambda = oracle.log_base(np.float32(rho * delta), delta, K)
        assert 0 < alpha < 1
        # level K-1 sits on the quantile: alpha^(K-1) = rho
        assert alpha ** (K - 1) == pytest.approx(rho, rel=5e-5)
        assert inv_lambda == pytest.approx(1 / math.log2(alpha), rel=1e-5)
        for r in np.float32(np.exp(rng.uniform(math.log(rho) * 1.3, 0, 20))).clip(0, 1):
            q = oracle.quant_log(float(r), inv_lambda, 0.0, K)
            t = math.log(float(r)) / math.log(alpha)
            d = np.abs(t - np.arange(K))
            if np.sort(d)[1] - np.sort(d)[0] > 1e-3:
                assert q == int(np.argmin(d)), (bits, alpha, r, q, t)
    # a zero among non-zeros takes the smallest level; the largest element takes level 0
    assert oracle.quant_log(0.0, -1.0, 0.0, K) == K - 1
    assert oracle.quant_log(1.0, -1.0, 0.49, K) == 0 and oracle.quant_log(1.0, -1.0, -0.49, K) == 0


def test_log_rounding_is_half_even_and_xi_shifts_it():
    # alpha = 1/2: log_alpha(r) = -log2(r); r = 2^-2.5 sits exactly between levels 2 and 3
    inv_lambda = -1.0
    r = float(np.float32(2.0 ** -2.5))
    t = -math.log2(r)
    assert abs(t - 2.5) < 1e-6
    assert oracle.quant_log(float(np.float32(2.0 ** -2.4)), inv_lambda, 0.0, 8) == 2
    assert oracle.quant_log(float(np.float32(2.0 ** -2.6)), inv_lambda, 0.0, 8) == 3
    assert oracle.quant_log(0.25, inv_lambda, 0.45, 8) == 2      # 2 + 0.45 -> 2
    assert oracle.quant_log(0.25, inv_lambda, 0.5, 8) == 2       # 2.5 -> 2 (ties to even)
    assert oracle.quant_log(0.125, inv_lambda, 0.5, 8) == 4      # 3.5 -> 4 (ties to even)
    assert oracle.quant_log(0.125, inv_lambda, -0.5, 8) == 2     # 2.5 -> 2
    assert oracle.quant_log(2.0 ** -20, inv_lambda, 0.0, 8) == 7  # clipped
    assert oracle.quant_log(2.0 ** -20, inv_lambda, 0.0, 256) == 20


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_roundtrip_invariants(bits):
    """dequant o quant o dequant = dequant; sign and zero behaviour of the signed quantizer."""
    y = oracle.codebook(oracle.DE_SIGNED, bits)
    K = len(y)
    for q in range(K):
        assert oracle.quant_nearest(y, float(y[q])) == q
    zero = int(np.where(y == 0)[0][0])
    assert oracle.quant_nearest(y, 0.0) == zero
    assert oracle.quant_nearest(y, 1.0) == K - 1 and y[K - 1] == 1.0
    assert oracle.quant_nearest(y, -1.0) == 0 and y[0] > -1.0          # no -1 level
    rng = np.random.default_rng(bits)
    for r in rng.uniform(-1, 1, 500).astype(np.float32):
        v = y[oracle.quant_nearest(y, float(r))]
        assert v == 0 or np.sign(v) == np.sign(r)
    # log levels: every code round-trips under xi = 0, and all levels are positive
    for alpha in (0.5, 0.9, 0.05, 0.999):
        if alpha ** (K - 1) < 2.0 ** -48:      # the base is clamped so that alpha^(K-1) >= 2^-48
            continue
        inv_lambda = 1.0 / oracle.log2_sp(alpha)
        for q in range(K):
            lv = oracle.pow_sm(alpha, q)
            assert lv > 0
            if lv >= 2.0 ** -100:
                assert oracle.quant_log(lv, inv_lambda, 0.0, K) == q, (alpha, q)


def test_pow_sm_is_a_product_chain():
    for alpha in (0.5, 0.75, 0.9990234375):
        for q in range(256):
            assert oracle.pow_sm(alpha, q) == pytest.approx(alpha ** q, rel=3e-6)
    a = np.float32(0.3)
    assert oracle.pow_sm(float(a), 3) == np.float32(a * np.float32(a * a))
    assert oracle.pow_sm(float(a), 0) == 1.0 and oracle.pow_sm(float(a), 1) == a


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_packed_layout_is_a_little_endian_bitstream(b):
    """Element e occupies bits [e*b, e*b+b) of the block's bytes read as one integer."""
    rng = np.random.default_rng(b)
    for block in (64, 128, 256):
        codes = rng.integers(0, 1 << b, block)
        buf = np.zeros(block * b // 8, np.uint8)
        for e, c in enumerate(codes):
            oracle.set_code(buf, e, b, int(c))
        big = int.from_bytes(buf.tobytes(), "little")
        for e, c in enumerate(codes):
            assert (big >> (e * b)) & ((1 << b) - 1) == c
            assert oracle.get_code(buf, e, b) == c
        # overwriting one element leaves its neighbours alone
        oracle.set_code(buf, 5, b, 0)
        assert oracle.get_code(buf, 4, b) == codes[4] and oracle.get_code(buf, 6, b) == codes[6]
    if b == 4:      # two per byte, low nibble first
        buf = np.zeros(1, np.uint8)
        oracle.set_code(buf, 0, 4, 0x3)
        oracle.set_code(buf, 1, 4, 0xA)
        assert buf[0] == 0xA3
    if b == 2:      # four per byte, lowest bits first
        buf = np.zeros(1, np.uint8)
        for e, c in enumerate((1, 2, 3, 0)):
            oracle.set_code(buf, e, 2, c)
        assert buf[0] == 0b00111001


def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 from the Random123 distribution (kat_vectors)."""
    kat = [
        ((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
        ((0xffffffff,) * 4, (0xffffffff,) * 2, (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
        ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
         (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1)),
    ]
    for ctr, key, out in kat:
        assert tuple(int(x) for x in oracle.philox4x32_10(ctr, key)) == out


def test_philox_draw_addressing_and_uniforms():
    """One Philox call serves eight elements; element idx takes halfword idx mod 8."""
    seed, step, tensor = 0x1234_5678_9ABC_DEF0, 7, 3
    for idx in (0, 1, 2, 3, 4, 5, 6, 7, 8, 13, (1 << 36) + 6, (1 << 36) + 7):
        words = oracle.philox4x32_10(
            ((idx >> 3) & 0xffffffff, (idx >> 3) >> 32, step, tensor * 4 + 1),
            (seed & 0xffffffff, seed >> 32))
        halves = [int(w) >> s & 0xffff for w in words for s in (0, 16)]
        assert oracle.philox_draw16(seed, step, tensor, idx, 1) == halves[idx & 7]
    # xi: midpoints of 2^16 cells of [-1/2, 1/2]: strictly inside, symmetric; u in [0, 1)
    assert oracle.xi(0) == -0.5 + 2.0 ** -17 and oracle.xi(0xffff) == 0.5 - 2.0 ** -17
    assert oracle.xi(0x8000) == 2.0 ** -17 and oracle.xi(0x7fff) == -(2.0 ** -17)
    for d in (0, 1, 0x1234, 0x7fff, 0xffff):
        assert oracle.xi(d) == -oracle.xi(0xffff - d)
        assert oracle.xi(d) == (d + 0.5) / 65536 - 0.5          # exact in binary32
    assert oracle.u01(0) == 0.0 and oracle.u01(0xffff) == 1.0 - 2.0 ** -16
    draws = [oracle.philox_draw16(1, 1, 0, i, 0) for i in range(4000)]
    xs = np.array([oracle.xi(d) for d in draws])
    assert abs(xs.mean()) < 0.02 and abs(xs.var() - 1 / 12) < 0.01
    assert len(set(draws)) > 3800                              # halves of a word are not copies


def test_log2_exp2_accuracy():
    rng = np.random.default_rng(0)
    xs = np.concatenate([np.exp2(rng.uniform(-100, 0, 4000)), 1 - np.exp2(rng.uniform(-24, -1, 500)),
                         np.exp2(rng.uniform(-1, 1, 500)), [1.0, 0.5, 2.0 ** -100, 0.70710677,
                                                            0.7071068, 1 - 2.0 ** -10]]).astype(np.float32)
    for x in xs:
        got, ref = oracle.log2_sp(float(x)), math.log2(float(x))
        assert abs(got - ref) <= 3e-7 * abs(ref) + 1e-37, (x, got, ref)
    assert oracle.log2_sp(1.0) == 0.0 and oracle.log2_sp(0.5) == -1.0 and oracle.log2_sp(0.25) == -2.0
    assert oracle.log2_sp(float(np.float32(1 - 2.0 ** -24))) < 0
    for x in np.concatenate([rng.uniform(-20, 0, 3000), -np.exp2(rng.uniform(-20, 0, 500)),
                             [0.0, -1.0, -0.5, -1.5]]).astype(np.float32):
        got, ref = oracle.exp2_sp(float(x)), 2.0 ** float(x)
        assert abs(got - ref) <= 1.5e-7 * ref, (x, got, ref)
    assert oracle.exp2_sp(0.0) == 1.0 and oracle.exp2_sp(-3.0) == 0.125


def test_stochastic_rounding_brackets():
    y = oracle.codebook(oracle.DE_SIGNED, 4)
    rng = np.random.default_rng(3)
    for r in rng.uniform(-1, 1, 300).astype(np.float32):
        lo = oracle.quant_stochastic(y, float(r), 0.999999)
        hi = oracle.quant_stochastic(y, float(r), 0.0)
        if r <= y[0]:
            assert lo == hi == 0
        else:
            assert hi == lo + 1 and y[lo] <= r <= y[hi]
            frac = (r - y[lo]) / (y[hi] - y[lo])
            assert oracle.quant_stochastic(y, float(r), float(frac) * 0.99) == hi
            assert oracle.quant_stochastic(y, float(r), min(float(frac) * 1.01 + 1e-6, 0.9999)) == lo
    for q in range(16):   # a value on a level stays there whatever u is
        assert oracle.quant_stochastic(y, float(y[q]), 0.5) == q


def test_bf16_stochastic_rounding_probabilities_are_exact():
    """Over all 2^16 draws the value goes to its upper bf16 neighbour exactly (dropped bits)
    times, so the mean over the draws is the value itself; representable values never move."""
    import struct
    vals = [1.0, 1.00001, -3.14159, 0.1, -1e-3, 7e-41, 65504.0, -0.0, 2.0 ** -126 * 1.5]
    for x in vals:
        bits = struct.unpack("<I", struct.pack("<f", x))[0]
        lo, hi = bits >> 16, bits & 0xffff
        got = np.array([oracle.bf16_sr(x, d) for d in range(0, 65536, 1 if hi in (0, 1) else 7)])
        assert set(np.unique(got)) <= {lo, lo + 1}
        if hi == 0:
            assert np.all(got == lo)                            # already bf16
        # every draw: up iff d >= 2^16 - dropped bits
        ds = np.arange(0, 65536, 1 if hi in (0, 1) else 7)
        assert np.array_equal(got == lo + 1, ds >= 65536 - hi)
    # counted in full for one value: ups == dropped bits, mean == value
    x = 1.2345678
    bits = struct.unpack("<I", struct.pack("<f", x))[0]
    got = np.array([oracle.bf16_sr(x, d) for d in range(65536)], dtype=np.int64)
    assert int((got == (bits >> 16) + 1).sum()) == bits & 0xffff
    as_float = np.array([struct.unpack("<f", struct.pack("<I", int(b) << 16))[0] for b in np.unique(got)])
    w = np.array([(got == b).sum() for b in np.unique(got)]) / 65536.0
    assert float((as_float.astype(np.float64) * w).sum()) == float(np.float32(x))
    # non-finite inputs are truncated, NaN stays NaN; the top finite bf16 binade can overflow
    assert oracle.bf16_sr(float("inf"), 0xffff) == 0x7f80 and oracle.bf16_sr(float("-inf"), 1) == 0xff80
    assert oracle.bf16_sr(float("nan"), 0) & 0x7fff > 0x7f80
    assert oracle.bf16_sr(3.4e38, 0xffff) == 0x7f80 and oracle.bf16_sr(3.4e38, 0) == 0x7f7f
    # nearest-even companion against torch
    import torch
    xs = np.random.default_rng(0).normal(0, 1, 2000).astype(np.float32)
    want = torch.from_numpy(xs).to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint16)
    assert [oracle.bf16_rn(float(v)) for v in xs] == [int(v) for v in want]
