"""slicemoe_pack on the GPU against the oracle: bit-exact scales, zero-points and both slice planes,
through the C ABI; plus the physical plane layout the header documents."""
import numpy as np
import pytest

from oracle import amat
from paper_2512_12990_b200 import synth

pytestmark = pytest.mark.gpu


def _pack_both(W, group, b_high=8, b_low=4):
    import torch
    from paper_2512_12990_b200 import binding as B
    N, K = W.shape
    pm = B.slicemoe_pack(torch.from_numpy(W).cuda(), group, b_high, b_low)
    msb = B.slicemoe_unpack_plane(pm.msb, N, K).cpu().numpy()
    lsb = B.slicemoe_unpack_plane(pm.lsb, N, K).cpu().numpy()
    s, z = B.slicemoe_unpack_meta(pm.scale, pm.zp, N, K, group)
    torch.cuda.synchronize()
    return pm, msb, lsb, s.cpu().numpy(), z.cpu().numpy()


def _check(W, group, b_high=8, b_low=4):
    o = amat.pack_matrix(W, group, b_high, b_low)
    pm, msb, lsb, s, z = _pack_both(W, group, b_high, b_low)
    assert np.array_equal(s.view(np.uint16), o["scale"].view(np.uint16)), "scale bits"
    assert np.array_equal(z, o["zp"]), "zero-points"
    assert np.array_equal(msb, o["msb"]), "MSB plane"
    assert np.array_equal(lsb, o["lsb"]), "LSB plane"
    assert np.array_equal((msb.astype(np.int32) << (b_high - b_low)) + lsb, o["q"])
    assert msb.max() < (1 << b_low) and lsb.max() < (1 << (b_high - b_low))
    return pm, o


@pytest.mark.parametrize("N,K,group", [
    (128, 256, 64), (256, 128, 64),              # tiny config matrices
    (1408, 2048, 128), (2048, 1408, 128),        # DeepSeek-V2-Lite / Qwen routed expert matrices
    (16, 128, 32), (48, 384, 32), (80, 640, 64), (16, 128, 128),   # single tile, ragged counts of tiles
])
def test_pack_bit_exact(N, K, group):
    W = synth.normal_f32(77, ("pack", N, K, group), (N, K), 0.02)
    _check(W, group)


@pytest.mark.parametrize("b_high,b_low", [(6, 3), (4, 2)])
@pytest.mark.parametrize("N,K,group", [(128, 256, 64), (1408, 2048, 128), (2048, 1408, 128), (48, 384, 32)])
def test_pack_bit_exact_narrower_slices(N, K, group, b_high, b_low):
    """MAT63 and MAT42 (Table 1): 6- and 4-bit codes, MSB slice = the top 3 / 2 bits, bit for bit the oracle's."""
    W = synth.normal_f32(79, ("pack", N, K, group, b_high), (N, K), 0.02)
    _check(W, group, b_high, b_low)
    # values that sit on the clamps and on rounding ties as well
    W2 = W.copy()
    W2[0, :8] = [0.0, 1.0, -1.0, 0.5, -0.5, 1e-8, 3.0, -3.0]
    _check(W2, group, b_high, b_low)


def test_pack_large_shared_expert_matrix():
    W = synth.normal_f32(78, ("pack-shared",), (5632, 2048), 0.02)
    _check(W, 128)


def test_pack_special_values():
    g = np.random.default_rng(5)
    W = (g.standard_normal((32, 512)) * 0.02).astype(np.float32)
    W[0, :128] = 0.0                        # degenerate: all zero
    W[1, :64] = 1e-12                       # scale underflows fp16
    W[2, :32] = 3.0e7                       # scale overflows fp16
    W[3, :128] = np.abs(W[3, :128])         # all positive: lo clamps to 0
    W[4, :128] = -np.abs(W[4, :128])        # all negative: hi clamps to 0
    W[5, 0:4] = [0.5, 1.5, 2.5, 3.5]        # ties once the scale is 1
    W[5, 4] = 255.0
    W[6, :] *= 1000.0                       # large magnitudes
    W[7, :] *= 1e-3                         # small magnitudes
    W[8, 5] = -0.0
    for group in (32, 64, 128):
        _check(W, group)


def test_constructive_round_trip_on_gpu():
    g = np.random.default_rng(9)
    group, N, K = 128, 32, 512
    ng = K // group
    s = (g.integers(128, 256, size=(N, ng)) * 2.0 ** (g.integers(-14, -3, size=(N, ng)) - 7.0)).astype(np.float16)
    zp = g.integers(0, 256, size=(N, ng)).astype(np.uint8)
    q = g.integers(0, 256, size=(N, ng, group)).astype(np.uint8)
    q[:, :, 0], q[:, :, 1] = 0, 255
    q = g.permuted(q, axis=2).reshape(N, K)
    W = (np.repeat(s.astype(np.float64), group, 1) * (q.astype(np.float64) - np.repeat(zp.astype(np.float64), group, 1))).astype(np.float32)
    _, msb, lsb, s2, z2 = _pack_both(W, group)
    assert np.array_equal(s2.view(np.uint16), s.view(np.uint16)) and np.array_equal(z2, zp)
    assert np.array_equal(msb.astype(np.int32) * 16 + lsb, q)


def test_physical_layout_matches_header():
    """Raw plane bytes against the layout written in slicemoe.h (re-derived here from that text)."""
    N, K, group = 48, 256, 64
    W = synth.normal_f32(79, ("layout",), (N, K), 0.02)
    pm, o = _check(W, group)
    raw = pm.msb.cpu().numpy().view("<u4")
    raw_s = pm.scale.cpu().numpy().view(np.uint16)
    raw_z = pm.zp.cpu().numpy()
    expect = np.zeros(N * K // 8, dtype=np.uint32)
    for rb in range(N // 16):
        for st in range(K // 64):
            for L in range(32):
                g, c = L // 4, L % 4
                for w in range(4):
                    word = 0
                    for j in range(4):
                        k = 64 * st + 16 * w + 4 * c + j
                        word |= int(o["msb"][16 * rb + g, k]) << (8 * j)
                        word |= int(o["msb"][16 * rb + g + 8, k]) << (8 * j + 4)
                    expect[((rb * (K // 64) + st) * 32 + L) * 4 + w] = word
    assert np.array_equal(raw, expect)
    ng = K // group
    es = np.zeros(N * ng, dtype=np.uint16)
    ez = np.zeros(N * ng, dtype=np.uint8)
    for n in range(N):
        for gidx in range(ng):
            es[((n // 16) * ng + gidx) * 16 + n % 16] = o["scale"].view(np.uint16)[n, gidx]
            ez[((n // 16) * ng + gidx) * 16 + n % 16] = o["zp"][n, gidx]
    assert np.array_equal(raw_s, es) and np.array_equal(raw_z, ez)


@pytest.mark.parametrize("b_high,b_low", [(4, 2), (6, 3), (8, 4)])
@pytest.mark.parametrize("N,K", [(16, 128), (48, 384), (1408, 2048)])
def test_dense_storage_of_narrow_slices(N, K, b_high, b_low):
    """slicemoe_compact_plane / _expand_plane: the plane's nibbles as the oracle's little-endian bit stream of
    b_low (MSB slice) and b_high - b_low (LSB slice) bits each, byte for byte, and back."""
    import torch
    from paper_2512_12990_b200 import binding as B
    W = synth.normal_f32(81, ("compact", N, K, b_high), (N, K), 0.02)
    pm = B.slicemoe_pack(torch.from_numpy(W).cuda(), 64 if K % 64 == 0 else 32, b_high, b_low)
    for plane, bits in ((pm.msb, b_low), (pm.lsb, b_high - b_low)):
        raw = plane.cpu().numpy().view(np.uint8).reshape(-1)
        nibbles = np.empty(raw.size * 2, dtype=np.uint8)
        nibbles[0::2], nibbles[1::2] = raw & 15, raw >> 4
        want = amat.compact_stream(nibbles[:8 * 4096], bits) if N * K > 8 * 4096 else amat.compact_stream(nibbles, bits)
        c = B.slicemoe_compact_plane(plane.view(torch.uint8), N, K, bits)
        got = c.cpu().numpy()
        assert got.size == N * K * bits // 8 == B.lib().slicemoe_compact_bytes(N, K, bits)
        assert np.array_equal(got[:want.size], want)
        if N * K > 8 * 4096:                      # the oracle is a plain loop: the large plane's tail too, in part
            tail = amat.compact_stream(nibbles[-8 * 1024:], bits)
            assert np.array_equal(got[-tail.size:], tail)
        back = B.slicemoe_expand_plane(c, N, K, bits)
        torch.cuda.synchronize()
        assert torch.equal(back, plane.view(torch.uint8).reshape(-1))
