"""Pins for oracle/amat.py: the AMAT format against what the paper's equation and the
arithmetic fix (exhaustive identities, hand examples, a constructive round trip, closed forms).
None of these re-types the oracle's own formula: each checks it from another side."""
import os

import numpy as np
import pytest

from oracle import amat

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "amat_hand_examples.txt")
MATS = [(8, 4), (6, 3), (4, 2)]


def _hand_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            left, right = line.split("|")
            bh, bl, q, zp, s = left.split()
            ql, lsb, zl, wh, wl = right.split()
            rows.append((int(bh), int(bl), int(q), int(zp), float(s), int(ql), int(lsb), int(zl),
                         float(wh), float(wl)))
    return rows


@pytest.mark.parametrize("bh,bl", MATS)
def test_truncation_is_msb_slice_exhaustive(bh, bl):
    """Truncating a b_high-bit code to its top b_low bits equals the stored MSB slice, and
    MSB+LSB reassembles the code (every code value)."""
    q = np.arange(1 << bh, dtype=np.uint8)
    msb, lsb = amat.slice_codes(q, bh, bl)
    shift = bh - bl
    assert np.array_equal(msb, q >> shift)                       # bit view of floor(q / 2^shift)
    assert np.array_equal(lsb, q & ((1 << shift) - 1))
    assert np.array_equal((msb.astype(int) << shift) | lsb, q)
    assert np.array_equal(amat.reassemble(msb, lsb, bh, bl), q)
    assert msb.max() == (1 << bl) - 1 and lsb.max() == (1 << shift) - 1
    # integer-division view, computed with Python ints
    assert [int(v) for v in msb] == [v // (2 ** shift) for v in range(1 << bh)]


@pytest.mark.parametrize("bh,bl", MATS)
def test_zero_point_truncation_exhaustive(bh, bl):
    zp = np.arange(1 << bh, dtype=np.uint8)
    zl = amat.truncate_zp(zp, bh, bl)
    assert [int(v) for v in zl] == [v // (2 ** (bh - bl)) for v in range(1 << bh)]


def test_hand_examples():
    rows = _hand_rows()
    assert len(rows) >= 10
    for bh, bl, q, zp, s, ql, lsb, zl, wh, wl in rows:
        qa = np.array([[q]], dtype=np.uint8)
        za = np.array([[zp]], dtype=np.uint8)
        sa = np.array([[s]], dtype=np.float16)
        m, l = amat.slice_codes(qa, bh, bl)
        assert (int(m[0, 0]), int(l[0, 0]), int(amat.truncate_zp(za, bh, bl)[0, 0])) == (ql, lsb, zl)
        s_used = float(sa[0, 0])                                  # the fp16 value of s
        hi = amat.dequant_high(sa, za, m, l, 1, bh, bl)[0, 0]
        lo = amat.dequant_low(sa, za, m, 1, bh, bl)[0, 0]
        assert hi == pytest.approx(wh * s_used / s, rel=1e-12, abs=1e-12)
        assert lo == pytest.approx(wl * s_used / s, rel=1e-12, abs=1e-12)


def test_low_bit_dequant_equals_brute_force_exhaustive():
    """(16 s)(q>>4 - zp>>4) == s ((q & 0xF0) - (zp & 0xF0)) for all 256 x 256 (q, zp) and a set of
    fp16 scales: the low-bit rule is the high-bit rule applied to code and zero-point with their
    low nibbles cleared.  The right-hand side is evaluated with Python floats, not the oracle."""
    q, zp = np.meshgrid(np.arange(256), np.arange(256), indexing="ij")
    q = q.reshape(1, -1).astype(np.uint8)
    zp = zp.reshape(1, -1).astype(np.uint8)
    msb, lsb = amat.slice_codes(q)
    for s in [1.0, 0.5, 0.0003662109375, 0.01, 6.1e-5, 123.5, 5.96e-8]:
        s16 = np.full(zp.shape, s, dtype=np.float16)
        sv = float(s16[0, 0])
        low = amat.dequant_low(s16, zp, msb, 1)
        brute = sv * ((q.astype(np.int64) & 0xF0) - (zp.astype(np.int64) & 0xF0)).astype(np.float64)
        assert np.array_equal(low, brute)
        # same thing through the high-bit rule with low nibbles forced to zero
        forced = amat.dequant_high(s16, zp & 0xF0, msb, np.zeros_like(lsb), 1)
        assert np.array_equal(low, forced)
        # slice identity: w8 - w4 = s ((q mod 16) - (zp mod 16)), so |w8 - w4| <= 15 s
        high = amat.dequant_high(s16, zp, msb, lsb, 1)
        diff = sv * ((q.astype(np.int64) & 15) - (zp.astype(np.int64) & 15)).astype(np.float64)
        assert np.allclose(high - low, diff, rtol=0, atol=1e-9 * sv)
        assert np.abs(high - low).max() <= 15 * sv * (1 + 1e-12)


@pytest.mark.parametrize("group", [32, 64, 128])
def test_quantiser_constructive_round_trip(group):
    """Draw (s, zp, q) with codes 0 and 255 present in every group, set W = s (q - zp) (exact in
    float32), and require quantize(W) to return exactly (s, zp, q)."""
    g = np.random.default_rng(7)
    N, K = 24, group * 5
    ng = K // group
    # fp16 scales with <= 8 significant bits so that 255*s and s*(q-zp) are exact in fp32
    mant = g.integers(128, 256, size=(N, ng)).astype(np.float64)
    expo = g.integers(-14, -3, size=(N, ng)).astype(np.float64)
    s = (mant * 2.0 ** (expo - 7)).astype(np.float16)
    assert np.array_equal(s.astype(np.float64), mant * 2.0 ** (expo - 7))
    zp = g.integers(0, 256, size=(N, ng)).astype(np.uint8)
    q = g.integers(0, 256, size=(N, ng, group)).astype(np.uint8)
    q[:, :, 0] = 0
    q[:, :, 1] = 255
    q = g.permuted(q, axis=2).reshape(N, K)
    W64 = np.repeat(s.astype(np.float64), group, 1) * (q.astype(np.float64) - np.repeat(zp.astype(np.float64), group, 1))
    W = W64.astype(np.float32)
    assert np.array_equal(W.astype(np.float64), W64)              # exactly representable
    s2, zp2, q2 = amat.quantize(W, group)
    assert np.array_equal(s2.view(np.uint16), s.view(np.uint16))
    assert np.array_equal(zp2, zp)
    assert np.array_equal(q2, q)
    # and the dequantised matrix is W again
    m, l = amat.slice_codes(q2)
    assert np.array_equal(amat.dequant_high(s2, zp2, m, l, group), W64)


def test_quantiser_error_bound_and_range():
    """For in-range data |w - w8| <= s/2 except at the clamped ends where it stays <= s."""
    g = np.random.default_rng(11)
    for group in (32, 64, 128):
        W = (g.standard_normal((64, group * 4)) * 0.02).astype(np.float32)
        W[3, :group] = np.abs(W[3, :group])            # all-positive group: lo clamps to 0
        W[5, :group] = -np.abs(W[5, :group])           # all-negative group
        p = amat.pack_matrix(W, group)
        w8 = amat.dequant_high(p["scale"], p["zp"], p["msb"], p["lsb"], group)
        s = np.repeat(p["scale"].astype(np.float64), group, 1)
        err = np.abs(W.astype(np.float64) - w8)
        assert (err <= s * (1 + 1e-6)).all()
        interior = (p["q"] > 0) & (p["q"] < 255)
        assert (err[interior] <= 0.5 * s[interior] * (1 + 1e-4)).all()
        assert np.mean(err <= 0.5 * s * (1 + 1e-4)) > 0.98
        # zero is representable: code zp dequantises to exactly 0
        assert p["zp"][3, 0] == 0 and p["zp"][5, 0] == 255


def test_quantiser_degenerate_groups():
    W = np.zeros((2, 64), dtype=np.float32)
    W[1, :32] = 1e-12                                   # scale underflows fp16 -> degenerate
    s, zp, q = amat.quantize(W, 32)
    assert (s == np.float16(1.0)).all() and (zp == 0).all() and (q == 0).all()
    W[0, :32] = 3.0e7                                   # (hi - lo)/255 overflows fp16 -> degenerate
    s, zp, q = amat.quantize(W, 32)
    assert s[0, 0] == np.float16(1.0) and zp[0, 0] == 0 and (q[0, :32] == 255).all()


def test_quantiser_rounding_half_even_and_scale_precision():
    """A plausible mistake (round-half-up, or quantising with the unrounded fp32 scale) changes
    these codes."""
    group = 32
    W = np.zeros((1, group), dtype=np.float32)
    W[0, 0] = 255.0                                     # hi = 255, lo = 0 -> s = 1, zp = 0
    W[0, 1:5] = [0.5, 1.5, 2.5, 3.5]                    # ties -> even: 0, 2, 2, 4
    s, zp, q = amat.quantize(W, group)
    assert s[0, 0] == np.float16(1.0) and zp[0, 0] == 0
    assert q[0, :5].tolist() == [255, 0, 2, 2, 4]
    # scale that is not an fp16 number: hi = 0.3 -> s32 = 0.3/255; codes must use float(fp16(s32))
    W = np.zeros((1, group), dtype=np.float32)
    W[0, 0] = 0.3
    W[0, 1] = 0.2
    s, zp, q = amat.quantize(W, group)
    s_used = np.float32(np.float16(np.float32(0.3) / np.float32(255)))
    assert s[0, 0] == np.float16(np.float32(0.3) / np.float32(255))
    assert q[0, 1] == int(np.rint(np.float32(0.2) / s_used))
    assert q[0, 0] == min(255, int(np.rint(np.float32(0.3) / s_used)))


def test_truncation_error_statistics_closed_form():
    """Low nibbles uniform on 0..15 and z = zp mod 16:  E[(w8 - w4)^2] = s^2 (21.25 + (7.5 - z)^2).
    Checked per z by enumeration of the 16 nibble values and on N(0, 0.02) weights at 5 %."""
    for z in range(16):
        vals = [(l - z) ** 2 for l in range(16)]
        assert sum(vals) / 16 == pytest.approx(21.25 + (7.5 - z) ** 2)
    g = np.random.default_rng(3)
    group = 128
    W = (g.standard_normal((256, 2048)) * 0.02).astype(np.float32)
    p = amat.pack_matrix(W, group)
    w8 = amat.dequant_high(p["scale"], p["zp"], p["msb"], p["lsb"], group)
    w4 = amat.dequant_low(p["scale"], p["zp"], p["msb"], group)
    s = np.repeat(p["scale"].astype(np.float64), group, 1)
    z = np.repeat((p["zp"] % 16).astype(np.float64), group, 1)
    measured = np.mean(((w8 - w4) / s) ** 2)
    predicted = np.mean(21.25 + (7.5 - z) ** 2)
    assert measured == pytest.approx(predicted, rel=0.05)
    # AMAT 4-bit error stays a small multiple of an independent 4-bit asymmetric quantiser's
    # (Table 1's qualitative claim), far from the failure of truncating codes alone.
    s4, zp4, q4 = amat.quantize(W, group, b_high=4)
    w4_base = np.repeat(s4.astype(np.float64), group, 1) * (q4.astype(np.float64) - np.repeat(zp4.astype(np.float64), group, 1))
    mse_amat = np.mean((W - w4) ** 2)
    mse_base = np.mean((W - w4_base) ** 2)
    assert 1.0 < mse_amat / mse_base < 3.5
    w4_codes_only = 16 * s * (p["msb"].astype(np.float64) - np.repeat(p["zp"].astype(np.float64), group, 1) / 16.0)
    # (keeping zp un-truncated happens to be unbiased per weight but is not what the paper
    # stores; the catastrophic variant drops the zero-point scaling altogether)
    w4_naive = 16 * s * (p["msb"].astype(np.float64) - np.repeat(p["zp"].astype(np.float64), group, 1))
    assert np.mean((W - w4_naive) ** 2) > 1e3 * mse_amat
    assert np.isfinite(w4_codes_only).all()


def test_canonical_nibble_packing():
    plane = np.array([[1, 2, 3, 4], [15, 0, 9, 7]], dtype=np.uint8)
    assert amat.nibble_pack_canonical(plane).tolist() == [0x21, 0x43, 0x0F, 0x79]


def test_compact_stream_is_the_little_endian_bit_stream():
    """Pins of the dense 2- / 3- / 4-bit slice storage: hand-worked bytes, the big-integer definition of a
    little-endian bit stream, and the round trip."""
    # 2 bits: values 1, 2, 3, 0 -> 0b00_11_10_01 = 0x39; then 3, 3, 3, 3 -> 0xff
    assert amat.compact_stream(np.array([1, 2, 3, 0, 3, 3, 3, 3]), 2).tolist() == [0x39, 0xFF]
    # 3 bits: 1, 2, 3, 4, 5, 6, 7, 0 -> bits 001 010 011 100 101 110 111 000 from the low end:
    # 1 + 2*8 + 3*64 + 4*512 + 5*4096 + 6*32768 + 7*262144 = 2,054,353 = 0x1F58D1 -> bytes d1 58 1f
    v = [1, 2, 3, 4, 5, 6, 7, 0]
    total = sum(x << (3 * i) for i, x in enumerate(v))
    assert total == 0x1F58D1
    assert amat.compact_stream(np.array(v), 3).tolist() == [0xD1, 0x58, 0x1F]
    # 4 bits is the nibble packing itself
    assert amat.compact_stream(np.array([1, 2, 3, 4, 15, 0, 9, 7]), 4).tolist() == [0x21, 0x43, 0x0F, 0x79]
    rng = np.random.default_rng(3)
    for bits in (2, 3, 4):
        vals = rng.integers(0, 1 << bits, 8 * 37).astype(np.uint8)
        s = amat.compact_stream(vals, bits)
        assert s.size == vals.size * bits // 8
        big = sum(int(x) << (bits * i) for i, x in enumerate(vals))
        assert bytes(s) == big.to_bytes(s.size, "little")
        assert np.array_equal(amat.compact_unstream(s, bits, vals.size), vals)
    with pytest.raises(AssertionError):
        amat.compact_stream(np.array([4, 0, 0, 0, 0, 0, 0, 0]), 2)      # does not fit 2 bits
