"""Oracle: AMAT weight format (Section 4.2 of the paper).  Test infrastructure only.

The paper gives the truncation rule (the displayed equation of Section 4.2):

    shift = b_high - b_low,  q_low = floor(q_high / 2^shift),  zp_low = floor(zp_high / 2^shift)

and says experts use grouped asymmetric integer quantisation (Table 1, footnote 1; Section
6.1).  It does not write the quantiser out; the reading used here is the standard affine
quantiser, stated step by step in `quantize`.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


def quantize(W: np.ndarray, group: int, b_high: int = 8):
    """Asymmetric per-group quantiser along K (Table 1 fn. 1 / Section 6.1: grouped asymmetric INT).

    W: float32 [N, K], K % group == 0.  Per row n and K-group g, in float32 arithmetic:
      lo = min(min_k w, 0), hi = max(max_k w, 0)
      s32 = (hi - lo) / qmax;  s16 = fp16_round_nearest_even(s32);  s = float32(s16)
      degenerate group (hi == lo, or s16 is 0 or inf): s16 = 1.0, zp = 0
      zp = clamp(rint(-lo / s), 0, qmax)
      q  = clamp(rint(w / s) + zp, 0, qmax)            (rint = round half to even)
    Returns (scale float16 [N, K/group], zp uint8 [N, K/group], q uint8 [N, K]).
    """
    W = np.asarray(W)
    assert W.dtype == np.float32 and W.ndim == 2
    N, K = W.shape
    assert K % group == 0
    qmax = (1 << b_high) - 1
    Wg = W.reshape(N, K // group, group)
    lo = np.minimum(Wg.min(axis=2), F32(0))
    hi = np.maximum(Wg.max(axis=2), F32(0))
    s32 = ((hi - lo) / F32(qmax)).astype(np.float32)
    with np.errstate(over="ignore"):
        s16 = s32.astype(np.float16)
    degenerate = (hi == lo) | (s16 == np.float16(0)) | ~np.isfinite(s16)
    s16 = np.where(degenerate, np.float16(1.0), s16).astype(np.float16)
    s = s16.astype(np.float32)
    zp_f = np.rint((-lo / s).astype(np.float32))
    zp = np.clip(zp_f, 0, qmax).astype(np.int32)
    zp = np.where(degenerate, 0, zp)
    r = np.rint((Wg / s[:, :, None]).astype(np.float32))
    r = np.clip(r, -1e9, 1e9).astype(np.int64)          # keep the integer add exact
    q = np.clip(r + zp[:, :, None], 0, qmax)
    return s16, zp.astype(np.uint8), q.reshape(N, K).astype(np.uint8)


def slice_codes(q: np.ndarray, b_high: int = 8, b_low: int = 4):
    """Split each b_high-bit code into its top b_low bits (MSB slice) and the remaining
    b_high - b_low bits (LSB slice), per the truncation rule of Section 4.2."""
    shift = b_high - b_low
    q = q.astype(np.int64)
    msb = q // (1 << shift)
    lsb = q - msb * (1 << shift)
    return msb.astype(np.uint8), lsb.astype(np.uint8)


def truncate_zp(zp: np.ndarray, b_high: int = 8, b_low: int = 4):
    """zp_low = floor(zp_high / 2^shift)  (Section 4.2).  Not stored; derived at use."""
    shift = b_high - b_low
    return (zp.astype(np.int64) // (1 << shift)).astype(np.uint8)


def reassemble(msb: np.ndarray, lsb: np.ndarray, b_high: int = 8, b_low: int = 4):
    """MSB slice and LSB slice together give back the b_high-bit code."""
    shift = b_high - b_low
    return (msb.astype(np.int64) * (1 << shift) + lsb.astype(np.int64)).astype(np.uint8)


def _expand(per_group: np.ndarray, group: int) -> np.ndarray:
    return np.repeat(per_group, group, axis=1)


def dequant_high(scale16, zp, msb, lsb, group: int, b_high: int = 8, b_low: int = 4) -> np.ndarray:
    """Full precision (both slices cached, Section 4.1): w = s * (q - zp), float64."""
    q = reassemble(msb, lsb, b_high, b_low).astype(np.float64)
    s = _expand(scale16.astype(np.float64), group)
    z = _expand(zp.astype(np.float64), group)
    return s * (q - z)


def dequant_low(scale16, zp, msb, group: int, b_high: int = 8, b_low: int = 4) -> np.ndarray:
    """MSB-only computation (Section 4.1) with the jointly truncated zero-point (Section 4.2):
    w = (2^shift * s) * (q_low - zp_low), float64.  The low-bit step is 2^shift high-bit steps,
    which keeps the low-bit quantiser on the same value range as the high-bit one."""
    shift = b_high - b_low
    s = _expand(scale16.astype(np.float64), group) * float(1 << shift)
    z = _expand(truncate_zp(zp, b_high, b_low).astype(np.float64), group)
    return s * (msb.astype(np.float64) - z)


def dequant(mat: dict, prec: int) -> np.ndarray:
    """mat: dict(scale, zp, msb, lsb, group[, b_high, b_low]); prec 1 = MSB+LSB, 0 = MSB only."""
    bh, bl = mat.get("b_high", 8), mat.get("b_low", 4)
    if prec:
        return dequant_high(mat["scale"], mat["zp"], mat["msb"], mat["lsb"], mat["group"], bh, bl)
    return dequant_low(mat["scale"], mat["zp"], mat["msb"], mat["group"], bh, bl)


def pack_matrix(W: np.ndarray, group: int, b_high: int = 8, b_low: int = 4) -> dict:
    """quantize + slice: the offline preparation of one weight matrix.

    Returns canonical (layout-free) arrays: scale fp16 [N, K/G], zp u8 [N, K/G],
    msb u8 [N, K] (values < 2^b_low), lsb u8 [N, K] (values < 2^(b_high-b_low))."""
    s16, zp, q = quantize(W, group, b_high)
    msb, lsb = slice_codes(q, b_high, b_low)
    return dict(scale=s16, zp=zp, msb=msb, lsb=lsb, q=q, group=group, b_high=b_high, b_low=b_low)


def nibble_pack_canonical(plane: np.ndarray) -> np.ndarray:
    """Canonical byte packing of a 4-bit plane [N, K] for dumps: byte (n*K + k)//2, even k in the
    low nibble."""
    flat = plane.reshape(-1).astype(np.uint8)
    assert flat.size % 2 == 0
    return (flat[0::2] | (flat[1::2] << 4)).astype(np.uint8)


def compact_stream(values: np.ndarray, bits: int) -> np.ndarray:
    """The dense storage of a slice narrower than a nibble (Table 1: MAT63 has 3-bit slices, MAT42 2-bit ones):
    a little-endian bit stream, value i in bits [i * bits, (i + 1) * bits).  values: 1-D, each < 2^bits, count a
    multiple of 8 (so the stream ends on a byte).  Returns uint8 [count * bits / 8]."""
    v = np.asarray(values, dtype=np.uint8).reshape(-1)
    assert bits in (2, 3, 4) and v.size % 8 == 0 and (v.size == 0 or int(v.max()) < (1 << bits))
    out = np.zeros(v.size * bits // 8, dtype=np.uint8)
    for i in range(v.size):                      # plain and slow on purpose
        pos = i * bits
        val = int(v[i]) << (pos & 7)
        out[pos >> 3] |= val & 0xFF
        if val >> 8:
            out[(pos >> 3) + 1] |= val >> 8
    return out


def compact_unstream(stream: np.ndarray, bits: int, count: int) -> np.ndarray:
    """Inverse of compact_stream: the first `count` values."""
    s = np.asarray(stream, dtype=np.uint8).reshape(-1)
    out = np.zeros(count, dtype=np.uint8)
    for i in range(count):
        pos = i * bits
        word = int(s[pos >> 3]) | (int(s[(pos >> 3) + 1]) << 8 if (pos >> 3) + 1 < s.size else 0)
        out[i] = (word >> (pos & 7)) & ((1 << bits) - 1)
    return out
