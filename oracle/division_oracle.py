"""CPU oracle for the DIVISION activation compress / decompress pair.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain NumPy statement of what the
method computes.  It exists so that the CUDA library can be checked element by element;
it is never a fallback.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import it; the CUDA package must not.

It shares no code, tables or constants with the CUDA path: both sides were written
separately from the same written definitions (the paper for the method; the "format"
notes below for what the paper leaves open).

What the method computes (DIVISION, Sec. 4.1 "Activation Map Compression" and Sec. 4.2
"Activation Map Decompression"; the forward and backward loops of Algorithm 1):

  compress    H^L = AveragePooling(H)            window = stride = B           (Sec. 4.1)
              H^H = H - UpSampling(H^L)          nearest interpolation         (Sec. 4.1)
              V^H = SR( (H^H - delta) / Delta )  Q-bit, stochastic rounding    (Eq. 9, "Quant")
              delta = min H^H, Delta = (max H^H - delta) / (2^Q - 1)
  decompress  H^H_hat = Delta * V^H + delta                                    (Sec. 4.2, Eq. 10)
              H_hat   = UpSampling(H^L) + H^H_hat                              (Sec. 4.2, Eq. 10)

Readings of points the paper leaves open (every one is also listed in the design notes):

  * quantisation group: one (delta, Delta) pair per sample (all C*H*W residuals of it); the
    variant with one bfloat16 pair per (sample, channel) plane, which is what the paper's byte
    count of Theorem 3A assumes, is stated in the last section of this file;
  * H or W not divisible by B: ceil grid, a partial tile is averaged over its in-bounds
    elements (this reproduces the paper's "N < B gives a 1x1 low-frequency map" rule);
  * the residual is taken against the STORED (rounded) low-frequency value, so that the
    decoder, which only has the stored value, reconstructs without a systematic bias;
  * stochastic rounding rounds UP with probability frac(t) (the paper's footnote states
    the two probabilities the other way round, which would contradict its own
    unbiasedness statement E[dequant(quant(h))] = h);
  * max == min inside a sample: Delta = 0, scale = 0, every code 0;
  * (delta, Delta) are kept in fp32;
  * arithmetic is IEEE fp32 (the paper's activations are fp32), one rounding per written
    operation, no fused multiply-add.

Format decisions of this build (the paper gives byte counts only):

  * random numbers: DIVRNG-v1, a stateless counter-based generator.  For sample n and
    in-sample flat index e = (c*H + h)*W + w:
        g = e >> 2
        z = seed XOR (0x9E3779B97F4A7C15 * (n + 1))          (all arithmetic mod 2^64)
        z = z + 0xD1B54A32D192ED03 * (g + 1)
        z ^= z >> 32;  z *= 0xD6E8FEB86659FD93
        z ^= z >> 32;  z *= 0xD6E8FEB86659FD93
        z ^= z >> 32
        field = (z >> (16 * (e & 3))) & 0xFFFF,   u = field * 2^-16   in [0, 1)
  * block-mean summation order (fp32): a tile is B x B values, positions outside the map
    count as +0.0; each tile column is summed down its B rows by a balanced pairwise tree
    (neighbours first; padded with +0.0 to the next power of two), then the B column sums
    are summed by the same tree; mean = sum / float(in-bounds count).  (For a full
    power-of-two tile of equal values every addition is then exact.)
  * packing: code of global flat element i = n*C*H*W + e goes to 32-bit word i // (32/Q),
    bit offset (i mod (32/Q)) * Q counted from the least significant bit; words are
    little-endian; unused high bits of the last word are zero;
  * blob: [lfc | pad to 128 B | packed words | pad to 128 B | stats (delta, Delta) * N].
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_MASK64 = (1 << 64) - 1
_K_SAMPLE = 0x9E3779B97F4A7C15
_K_GROUP = 0xD1B54A32D192ED03
_K_MIX = 0xD6E8FEB86659FD93

F32 = "f32"
BF16 = "bf16"
_DTYPE_BYTES = {F32: 4, BF16: 2}
SECTION_ALIGN = 128
SUPPORTED_QBITS = (1, 2, 4, 8)


# ----------------------------------------------------------------------------------------
# bfloat16 <-> float32 (bit patterns; round-to-nearest-even)
# ----------------------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    return ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to fp32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(a32: np.ndarray, dtype: str) -> np.ndarray:
    """Value of `a32` after being stored in `dtype`, returned as fp32."""
    if dtype == F32:
        return np.asarray(a32, dtype=np.float32)
    if dtype == BF16:
        return bf16_bits_to_f32(f32_to_bf16_bits(a32))
    raise ValueError(f"unknown dtype {dtype!r}")


def widen_input(x: np.ndarray, x_dtype: str) -> np.ndarray:
    """fp32 view of the activation map: fp32 arrays pass through, bf16 arrives as uint16 bits."""
    if x_dtype == F32:
        if x.dtype != np.float32:
            raise TypeError("fp32 activation map expected as a float32 array")
        return x
    if x_dtype == BF16:
        if x.dtype != np.uint16:
            raise TypeError("bf16 activation map expected as uint16 bit patterns")
        return bf16_bits_to_f32(x)
    raise ValueError(f"unknown dtype {x_dtype!r}")


# ----------------------------------------------------------------------------------------
# sizes (closed form of the compressed representation)
# ----------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Layout:
    lfc_off: int
    lfc_bytes: int
    packed_off: int
    packed_bytes: int
    stats_off: int
    stats_bytes: int
    total_bytes: int          # blob size including alignment padding
    closed_form_bytes: int    # lfc + packed + stats without padding
    raw_bytes: int            # N*C*H*W*sizeof(x)


def _align(v: int, a: int) -> int:
    return (v + a - 1) // a * a


def grid_shape(h: int, w: int, block: int) -> tuple[int, int]:
    """Low-frequency map size: ceil grid (a side shorter than B gives one tile, Sec. 4.1 footnote)."""
    return -(-h // block), -(-w // block)


def compressed_layout(n: int, c: int, h: int, w: int, block: int, qbits: int,
                      x_dtype: str = F32, lfc_dtype: str = F32) -> Layout:
    """Bytes of the cached tuple (H^L, V^H, Delta, delta) of Sec. 4.1, in this build's blob layout.

    closed form = N*C*ceil(H/B)*ceil(W/B)*sizeof(lfc) + ceil(N*C*H*W*Q/32)*4 + 8*N.
    """
    if min(n, c, h, w) < 1 or block < 1 or qbits not in SUPPORTED_QBITS:
        raise ValueError("bad descriptor")
    hb, wb = grid_shape(h, w, block)
    lfc_bytes = n * c * hb * wb * _DTYPE_BYTES[lfc_dtype]
    packed_bytes = -(-(n * c * h * w * qbits) // 32) * 4
    stats_bytes = 8 * n
    packed_off = _align(lfc_bytes, SECTION_ALIGN)
    stats_off = _align(packed_off + packed_bytes, SECTION_ALIGN)
    return Layout(0, lfc_bytes, packed_off, packed_bytes, stats_off, stats_bytes,
                  stats_off + stats_bytes, lfc_bytes + packed_bytes + stats_bytes,
                  n * c * h * w * _DTYPE_BYTES[x_dtype])


def paper_conv_block_rate(side: int, block: int, qbits: int) -> float:
    """Compression rate of one conv-BN-ReLU block with the PAPER's byte accounting (Theorem 3A proof).

    Per channel plane of side*side fp32 values: normal training caches 4*side^2 bytes for the
    conv and for the BN layer and side^2 bytes for ReLU; DIVISION caches, for conv and BN each,
    a bf16 low-frequency map, Q bits per element and 4 bytes of (Delta, delta), plus one bit per
    element for ReLU.  Written from the byte counts, not from the theorem's closed formula.
    """
    n2 = side * side
    normal = 4 * n2 * 2 + n2
    lfc = 2.0 * n2 / min(block * block, n2)
    hfc = qbits * n2 / 8.0
    division = (lfc + hfc + 4.0) * 2 + n2 / 8.0
    return normal / division


# ----------------------------------------------------------------------------------------
# DIVRNG-v1
# ----------------------------------------------------------------------------------------
def divrng_fields(seed: int, n: int, e: np.ndarray) -> np.ndarray:
    """16-bit random fields for sample `n` at in-sample flat indices `e` (format notes above)."""
    e = np.asarray(e, dtype=np.uint64)
    g = e >> np.uint64(2)
    z0 = (int(seed) & _MASK64) ^ ((_K_SAMPLE * (int(n) + 1)) & _MASK64)
    with np.errstate(over="ignore"):
        z = np.uint64(z0) + np.uint64(_K_GROUP) * (g + np.uint64(1))
        z ^= z >> np.uint64(32)
        z *= np.uint64(_K_MIX)
        z ^= z >> np.uint64(32)
        z *= np.uint64(_K_MIX)
        z ^= z >> np.uint64(32)
    shift = (e & np.uint64(3)) * np.uint64(16)
    return ((z >> shift) & np.uint64(0xFFFF)).astype(np.uint16)


# ----------------------------------------------------------------------------------------
# low-frequency component
# ----------------------------------------------------------------------------------------
def _tiles(x32: np.ndarray, block: int):
    """View the map as tiles: returns (t, rows, cols) with t[N,C,Hb,Wb,B,B] zero-padded."""
    n, c, h, w = x32.shape
    hb, wb = grid_shape(h, w, block)
    xp = np.zeros((n, c, hb * block, wb * block), dtype=x32.dtype)
    xp[:, :, :h, :w] = x32
    t = xp.reshape(n, c, hb, block, wb, block).transpose(0, 1, 2, 4, 3, 5)
    rows = np.minimum(block, h - np.arange(hb) * block)      # in-bounds rows of tile row bh
    cols = np.minimum(block, w - np.arange(wb) * block)      # in-bounds cols of tile col bw
    return t, rows, cols


def _pairwise_tree_sum(a: np.ndarray, axis: int) -> np.ndarray:
    """Balanced pairwise sum along `axis` (neighbours first), zero-padded to a power of two."""
    a = np.moveaxis(a, axis, -1)
    width = 1
    while width < a.shape[-1]:
        width *= 2
    if width != a.shape[-1]:
        pad = np.zeros(a.shape[:-1] + (width - a.shape[-1],), dtype=a.dtype)
        a = np.concatenate([a, pad], axis=-1)
    while a.shape[-1] > 1:
        a = a[..., 0::2] + a[..., 1::2]
    return a[..., 0]


def lfc_mean_f32(x32: np.ndarray, block: int) -> np.ndarray:
    """H^L = AveragePooling(H), window = stride = B (Sec. 4.1), in fp32 with the build's summation order."""
    t, rows, cols = _tiles(np.asarray(x32, dtype=np.float32), block)   # t[..., row, col], zeros outside
    colsum = _pairwise_tree_sum(t, axis=-2)          # down the rows of every tile column
    total = _pairwise_tree_sum(colsum, axis=-1)      # across the column sums
    count = (rows[:, None] * cols[None, :]).astype(np.float32)
    return (total / count[None, None]).astype(np.float32)


def lfc_mean_f64(x: np.ndarray, block: int) -> np.ndarray:
    """The same block mean by its plain definition in fp64 (no prescribed order)."""
    t, rows, cols = _tiles(np.asarray(x, dtype=np.float64), block)
    count = (rows[:, None] * cols[None, :]).astype(np.float64)
    return t.sum(axis=(-1, -2)) / count[None, None]


def upsample_nearest(lfc: np.ndarray, block: int, h: int, w: int) -> np.ndarray:
    """UpSampling(H^L): element (h, w) takes the value of tile (h // B, w // B) (Sec. 4.1)."""
    up = np.repeat(np.repeat(lfc, block, axis=2), block, axis=3)
    return up[:, :, :h, :w]


# ----------------------------------------------------------------------------------------
# quantiser (Eq. 9) and its inverse
# ----------------------------------------------------------------------------------------
def sample_stats(r_flat: np.ndarray, qbits: int):
    """delta = min, Delta = (max - min)/(2^Q - 1), scale = (2^Q - 1)/(max - min) of one sample."""
    qmax = np.float32((1 << qbits) - 1)
    delta = np.float32(r_flat.min())
    top = np.float32(r_flat.max())
    rng = np.float32(top - delta)
    if rng > 0:
        with np.errstate(over="ignore", divide="ignore"):
            scale = np.float32(qmax / rng)
            step = np.float32(rng / qmax)
        if not np.isfinite(scale):
            scale, step = np.float32(0), np.float32(0)
    else:
        scale, step = np.float32(0), np.float32(0)
    return delta, step, scale


def quantize(r_flat: np.ndarray, delta: np.float32, scale: np.float32, fields: np.ndarray,
             qbits: int) -> np.ndarray:
    """V^H = floor(t) + [u < frac(t)], t = (H^H - delta) * scale, clamped to [0, 2^Q - 1]  (Eq. 9)."""
    r_flat = np.asarray(r_flat, dtype=np.float32)
    t = (r_flat - np.float32(delta)) * np.float32(scale)      # two fp32 roundings
    f = np.floor(t)
    p = t - f                                                  # exact
    u = fields.astype(np.float32) * np.float32(2.0 ** -16)     # exact
    code = f.astype(np.int64) + (u < p)
    return np.clip(code, 0, (1 << qbits) - 1).astype(np.uint8)


def dequantize(codes: np.ndarray, delta: np.float32, step: np.float32) -> np.ndarray:
    """H^H_hat = Delta * V^H + delta (Sec. 4.2): one fp32 multiply, then one fp32 add."""
    return np.float32(step) * codes.astype(np.float32) + np.float32(delta)


# ----------------------------------------------------------------------------------------
# bit packing
# ----------------------------------------------------------------------------------------
def pack_codes(codes_flat: np.ndarray, qbits: int) -> np.ndarray:
    """Q-bit codes in flat element order -> little-endian 32-bit words, low bits first."""
    per = 32 // qbits
    total = codes_flat.size
    nwords = -(-total // per)
    padded = np.zeros(nwords * per, dtype=np.uint32)
    padded[:total] = codes_flat
    shifts = (np.arange(per, dtype=np.uint32) * np.uint32(qbits))
    return np.bitwise_or.reduce(padded.reshape(nwords, per) << shifts[None, :], axis=1).astype(np.uint32)


def unpack_codes(words: np.ndarray, qbits: int, total: int) -> np.ndarray:
    per = 32 // qbits
    shifts = (np.arange(per, dtype=np.uint32) * np.uint32(qbits))
    codes = (words.astype(np.uint32)[:, None] >> shifts[None, :]) & np.uint32((1 << qbits) - 1)
    return codes.reshape(-1)[:total].astype(np.uint8)


# ----------------------------------------------------------------------------------------
# the pair
# ----------------------------------------------------------------------------------------
@dataclass
class Compressed:
    shape: tuple
    block: int
    qbits: int
    x_dtype: str
    lfc_dtype: str
    lfc: np.ndarray        # [N,C,Hb,Wb] fp32 VALUES as stored (already rounded to lfc_dtype)
    codes: np.ndarray      # [N, C*H*W] uint8
    words: np.ndarray      # packed uint32 words
    delta: np.ndarray      # [N] fp32
    step: np.ndarray       # [N] fp32  (Delta)
    layout: Layout

    def blob(self) -> np.ndarray:
        """The compressed buffer exactly as the library lays it out (padding bytes zero)."""
        out = np.zeros(self.layout.total_bytes, dtype=np.uint8)
        if self.lfc_dtype == F32:
            lfc_raw = self.lfc.astype("<f4").tobytes()
        else:
            lfc_raw = f32_to_bf16_bits(self.lfc).astype("<u2").tobytes()
        lo = self.layout
        out[lo.lfc_off:lo.lfc_off + lo.lfc_bytes] = np.frombuffer(lfc_raw, dtype=np.uint8)
        out[lo.packed_off:lo.packed_off + lo.packed_bytes] = np.frombuffer(
            self.words.astype("<u4").tobytes(), dtype=np.uint8)
        stats = np.stack([self.delta, self.step], axis=1).astype("<f4")
        out[lo.stats_off:lo.stats_off + lo.stats_bytes] = np.frombuffer(stats.tobytes(), dtype=np.uint8)
        return out


def compress(x: np.ndarray, block: int, qbits: int, seed: int,
             x_dtype: str = F32, lfc_dtype: str = F32, first_sample: int = 0) -> Compressed:
    """Forward-loop steps of Algorithm 1 (pooling, residual, Quant, cache) for one activation map H of shape N x C x H x W.

    `first_sample`: x holds samples first_sample, first_sample+1, ... of a larger mini-batch (samples
    are independent, so a slice of a batch can be checked alone; only the random stream depends on
    the sample's index in the batch).
    """
    if qbits not in SUPPORTED_QBITS:
        raise ValueError("Q must divide 32")
    x32 = widen_input(x, x_dtype)
    n, c, h, w = x32.shape
    chw = c * h * w
    lfc = round_to_dtype(lfc_mean_f32(x32, block), lfc_dtype)           # AveragePooling (+ storage rounding)
    r = (x32 - upsample_nearest(lfc, block, h, w)).reshape(n, chw)       # residual, one fp32 rounding
    codes = np.empty((n, chw), dtype=np.uint8)
    delta = np.empty(n, dtype=np.float32)
    step = np.empty(n, dtype=np.float32)
    e = np.arange(chw, dtype=np.uint64)
    for i in range(n):                                                   # Quant, per sample
        delta[i], step[i], scale = sample_stats(r[i], qbits)
        codes[i] = quantize(r[i], delta[i], scale, divrng_fields(seed, first_sample + i, e), qbits)
    words = pack_codes(codes.reshape(-1), qbits)
    layout = compressed_layout(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    return Compressed((n, c, h, w), block, qbits, x_dtype, lfc_dtype, lfc, codes, words, delta, step, layout)


def decompress(comp: Compressed) -> np.ndarray:
    """Backward-loop steps of Algorithm 1 (Dequant, up-sample and add); returns fp32 values, already rounded to the activation dtype."""
    n, c, h, w = comp.shape
    codes = unpack_codes(comp.words, comp.qbits, n * c * h * w).reshape(n, c * h * w)
    hh = np.empty((n, c * h * w), dtype=np.float32)
    for i in range(n):
        hh[i] = dequantize(codes[i], comp.delta[i], comp.step[i])
    xhat = upsample_nearest(comp.lfc, comp.block, h, w) + hh.reshape(n, c, h, w)
    return round_to_dtype(xhat.astype(np.float32), comp.x_dtype)


def parse_blob(blob: np.ndarray, n: int, c: int, h: int, w: int, block: int, qbits: int,
               x_dtype: str = F32, lfc_dtype: str = F32) -> Compressed:
    """Read a compressed buffer (for instance one the CUDA library wrote) back into its parts."""
    lo = compressed_layout(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    hb, wb = grid_shape(h, w, block)
    raw = blob[lo.lfc_off:lo.lfc_off + lo.lfc_bytes]
    if lfc_dtype == F32:
        lfc = raw.view("<f4").astype(np.float32)
    else:
        lfc = bf16_bits_to_f32(raw.view("<u2"))
    lfc = lfc.reshape(n, c, hb, wb)
    words = blob[lo.packed_off:lo.packed_off + lo.packed_bytes].view("<u4").astype(np.uint32)
    stats = blob[lo.stats_off:lo.stats_off + lo.stats_bytes].view("<f4").reshape(n, 2)
    codes = unpack_codes(words, qbits, n * c * h * w).reshape(n, c * h * w)
    return Compressed((n, c, h, w), block, qbits, x_dtype, lfc_dtype, lfc, codes, words,
                      stats[:, 0].copy(), stats[:, 1].copy(), lo)


# ----------------------------------------------------------------------------------------
# per-plane quantisation groups with bfloat16 (delta, Delta)
# ----------------------------------------------------------------------------------------
# The paper counts N^2*Q/8 + 4 bytes per channel plane for the high-frequency component
# (proof of Theorem 3A) and says that Delta and delta are cached in bfloat16 (Sec. 4.1): one
# (delta, Delta) pair of two bfloat16 numbers per (sample, channel) plane.  This section states
# that variant.  Everything else (pooling, residual against the stored low-frequency value,
# stochastic rounding, DIVRNG-v1, packing order) is as above.
#
# Reading for the bfloat16 rounding, on which the paper is silent: a delta rounded to NEAREST
# could land above the true minimum and make (h - delta)/Delta negative, and a Delta rounded
# down could push the largest code past 2^Q - 1.  So
#     delta_b = the largest bfloat16 number <= min H^H          (rounded down)
#     Delta_b = the smallest bfloat16 number >= (max H^H - delta_b) / (2^Q - 1)   (rounded up)
# and both the encoder and the decoder use exactly these stored numbers:
#     t = (h - delta_b) * (1 / Delta_b),   h_hat = Delta_b * code + delta_b.
# Then 0 <= t <= (2^Q - 1) up to fp32 rounding (the clamp of Eq. 9's range only absorbs that),
# |h_hat - h| <= Delta_b, and E[h_hat] = h as in Sec. 4.1.  A zero is stored as +0.0.  A plane whose
# Delta_b or 1/Delta_b is zero or not finite is degenerate: Delta_b = 0 is stored, every code is 0
# (and delta_b = 0 too when the minimum lies below the most negative finite bfloat16 number).
def bf16_floor_bits(a: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns of the largest bfloat16 numbers <= a (finite fp32 input)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    hi = u >> np.uint64(16)
    inexact = (u & np.uint64(0xFFFF)) != 0
    hi = hi + (inexact & (a < 0)).astype(np.uint64)      # truncation moves a negative number up
    hi = np.where(a == 0, np.uint64(0), hi)
    return hi.astype(np.uint16)


def bf16_ceil_bits(a: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns of the smallest bfloat16 numbers >= a (finite fp32 input)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    hi = u >> np.uint64(16)
    inexact = (u & np.uint64(0xFFFF)) != 0
    hi = hi + (inexact & (a > 0)).astype(np.uint64)      # truncation moves a positive number down
    hi = np.where(a == 0, np.uint64(0), hi)
    return hi.astype(np.uint16)


def plane_stats(r_plane: np.ndarray, qbits: int):
    """(delta_b, Delta_b, scale) of one (sample, channel) plane, all as fp32 values (rule above)."""
    qmax = np.float32((1 << qbits) - 1)
    low = np.float32(r_plane.min())
    top = np.float32(r_plane.max())
    delta_b = bf16_bits_to_f32(bf16_floor_bits(np.array([low])))[0]
    zero = np.float32(0)
    if not np.isfinite(delta_b):                       # minimum below the most negative bfloat16 number
        return zero, zero, zero
    with np.errstate(over="ignore", divide="ignore", invalid="ignore"):
        rng = np.float32(top - delta_b)
        step = np.float32(rng / qmax)
        step_b = bf16_bits_to_f32(bf16_ceil_bits(np.array([step])))[0] if np.isfinite(step) else np.float32(np.inf)
        scale = np.float32(np.float32(1) / step_b) if step_b > 0 else zero
    if not (np.isfinite(step_b) and step_b > 0 and np.isfinite(scale) and scale > 0):
        return delta_b, zero, zero
    return delta_b, step_b, scale


def plane_layout(n: int, c: int, h: int, w: int, block: int, qbits: int,
                 x_dtype: str = F32, lfc_dtype: str = F32) -> Layout:
    """As compressed_layout, but the stats section holds N*C pairs of bfloat16: 4 bytes per plane."""
    lo = compressed_layout(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    stats_bytes = 4 * n * c
    return Layout(lo.lfc_off, lo.lfc_bytes, lo.packed_off, lo.packed_bytes, lo.stats_off, stats_bytes,
                  lo.stats_off + stats_bytes, lo.lfc_bytes + lo.packed_bytes + stats_bytes, lo.raw_bytes)


@dataclass
class PlaneCompressed:
    shape: tuple
    block: int
    qbits: int
    x_dtype: str
    lfc_dtype: str
    lfc: np.ndarray        # [N,C,Hb,Wb] fp32 values as stored
    codes: np.ndarray      # [N, C, H*W] uint8
    words: np.ndarray      # packed uint32 words (same element order as the per-sample form)
    delta: np.ndarray      # [N, C] fp32 values of the stored bfloat16 delta_b
    step: np.ndarray       # [N, C] fp32 values of the stored bfloat16 Delta_b
    layout: Layout

    def blob(self) -> np.ndarray:
        out = np.zeros(self.layout.total_bytes, dtype=np.uint8)
        if self.lfc_dtype == F32:
            lfc_raw = self.lfc.astype("<f4").tobytes()
        else:
            lfc_raw = f32_to_bf16_bits(self.lfc).astype("<u2").tobytes()
        lo = self.layout
        out[lo.lfc_off:lo.lfc_off + lo.lfc_bytes] = np.frombuffer(lfc_raw, dtype=np.uint8)
        out[lo.packed_off:lo.packed_off + lo.packed_bytes] = np.frombuffer(
            self.words.astype("<u4").tobytes(), dtype=np.uint8)
        pair = np.stack([f32_to_bf16_bits(self.delta.reshape(-1)),       # exact: the values are bfloat16
                         f32_to_bf16_bits(self.step.reshape(-1))], axis=1).astype("<u2")
        out[lo.stats_off:lo.stats_off + lo.stats_bytes] = np.frombuffer(pair.tobytes(), dtype=np.uint8)
        return out


def compress_planes(x: np.ndarray, block: int, qbits: int, seed: int,
                    x_dtype: str = F32, lfc_dtype: str = F32, first_sample: int = 0) -> PlaneCompressed:
    """The forward-loop steps of Algorithm 1 with one quantisation group per (sample, channel) plane."""
    if qbits not in SUPPORTED_QBITS:
        raise ValueError("Q must divide 32")
    x32 = widen_input(x, x_dtype)
    n, c, h, w = x32.shape
    hw = h * w
    lfc = round_to_dtype(lfc_mean_f32(x32, block), lfc_dtype)
    r = (x32 - upsample_nearest(lfc, block, h, w)).reshape(n, c, hw)
    codes = np.empty((n, c, hw), dtype=np.uint8)
    delta = np.empty((n, c), dtype=np.float32)
    step = np.empty((n, c), dtype=np.float32)
    for i in range(n):
        fields = divrng_fields(seed, first_sample + i, np.arange(c * hw, dtype=np.uint64)).reshape(c, hw)
        for j in range(c):                                               # Quant, per plane
            delta[i, j], step[i, j], scale = plane_stats(r[i, j], qbits)
            codes[i, j] = quantize(r[i, j], delta[i, j], scale, fields[j], qbits)
    words = pack_codes(codes.reshape(-1), qbits)
    layout = plane_layout(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    return PlaneCompressed((n, c, h, w), block, qbits, x_dtype, lfc_dtype, lfc, codes, words, delta, step, layout)


def decompress_planes(comp: PlaneCompressed) -> np.ndarray:
    """The backward-loop steps of Algorithm 1 for per-plane groups; fp32 values rounded to the activation dtype."""
    n, c, h, w = comp.shape
    codes = unpack_codes(comp.words, comp.qbits, n * c * h * w).reshape(n, c, h * w)
    hh = (comp.step[:, :, None].astype(np.float32) * codes.astype(np.float32)
          + comp.delta[:, :, None].astype(np.float32)).astype(np.float32)
    xhat = upsample_nearest(comp.lfc, comp.block, h, w) + hh.reshape(n, c, h, w)
    return round_to_dtype(xhat.astype(np.float32), comp.x_dtype)


def parse_plane_blob(blob: np.ndarray, n: int, c: int, h: int, w: int, block: int, qbits: int,
                     x_dtype: str = F32, lfc_dtype: str = F32) -> PlaneCompressed:
    """Read a per-plane compressed buffer back into its parts."""
    lo = plane_layout(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    hb, wb = grid_shape(h, w, block)
    raw = blob[lo.lfc_off:lo.lfc_off + lo.lfc_bytes]
    lfc = raw.view("<f4").astype(np.float32) if lfc_dtype == F32 else bf16_bits_to_f32(raw.view("<u2"))
    lfc = lfc.reshape(n, c, hb, wb)
    words = blob[lo.packed_off:lo.packed_off + lo.packed_bytes].view("<u4").astype(np.uint32)
    pair = blob[lo.stats_off:lo.stats_off + lo.stats_bytes].view("<u2").reshape(n, c, 2)
    codes = unpack_codes(words, qbits, n * c * h * w).reshape(n, c, h * w)
    return PlaneCompressed((n, c, h, w), block, qbits, x_dtype, lfc_dtype, lfc, codes, words,
                           bf16_bits_to_f32(pair[:, :, 0].copy()), bf16_bits_to_f32(pair[:, :, 1].copy()), lo)


# ----------------------------------------------------------------------------------------
# ReLU and dropout operators with a packed 1-bit mask (the paper's appendix algorithms
# "Relu operator" and "Dropout operator"; 1 bit per element in the byte count of Theorem 3A)
# ----------------------------------------------------------------------------------------
# Forward:  V = mask, H_out = V (.) H_in, V packed and cached.   Backward:  grad_in = V (.) grad_out.
# Readings:
#   * ReLU: the paper writes V = sgn(H); for ReLU this is read as the indicator of H > 0 (so that V (.) H is
#     max(H, 0)); zeros of either sign and NaN give V = 0;
#   * dropout: V = 1 (keep) with probability 1 - p, p = drop_threshold / 65536; element i is dropped iff its
#     16-bit DIVRNG-v1 field (sample index 0, flat index i) is < drop_threshold.  As in the paper's algorithm
#     there is no 1/(1-p) rescaling;
#   * "(.)" with a 0/1 mask is a select: a masked position is +0.0 (inputs are finite);
#   * packing: bit (i mod 32) of little-endian 32-bit word i // 32, unused high bits of the last word zero
#     (the Q = 1 case of the packing rule above).
def mask_bytes(total: int) -> int:
    """Bytes of the packed mask of `total` elements: whole 32-bit words."""
    return -(-int(total) // 32) * 4


def pack_mask(v_flat: np.ndarray) -> np.ndarray:
    return pack_codes(np.asarray(v_flat, dtype=np.uint8).reshape(-1), 1)


def unpack_mask(words: np.ndarray, total: int) -> np.ndarray:
    return unpack_codes(words, 1, total)


def relu_forward(x: np.ndarray, x_dtype: str = F32):
    """Forward of the "Relu operator": returns (H_out as fp32 values, packed mask words)."""
    x32 = widen_input(x, x_dtype).reshape(-1)
    v = (x32 > 0).astype(np.uint8)
    out = np.where(v == 1, x32, np.float32(0)).astype(np.float32)
    return out, pack_mask(v)


def dropout_forward(x: np.ndarray, seed: int, drop_threshold: int, x_dtype: str = F32):
    """Forward of the "Dropout operator" (no rescaling): returns (H_out as fp32 values, packed mask words)."""
    if not 0 <= int(drop_threshold) <= 65536:
        raise ValueError("drop_threshold must lie in [0, 65536]")
    x32 = widen_input(x, x_dtype).reshape(-1)
    fields = divrng_fields(seed, 0, np.arange(x32.size, dtype=np.uint64)).astype(np.uint32)
    v = (fields >= np.uint32(drop_threshold)).astype(np.uint8)
    out = np.where(v == 1, x32, np.float32(0)).astype(np.float32)
    return out, pack_mask(v)


def mask_backward(words: np.ndarray, grad_out: np.ndarray, x_dtype: str = F32) -> np.ndarray:
    """Backward of both operators: grad_in = V (.) grad_out, as fp32 values."""
    g32 = widen_input(grad_out, x_dtype).reshape(-1)
    v = unpack_mask(words, g32.size)
    return np.where(v == 1, g32, np.float32(0)).astype(np.float32)


# ----------------------------------------------------------------------------------------
# 1-D activation maps  (appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N,
# average pooling and nearest up-sampling along the last axis, Quant and its inverse unchanged)
# ----------------------------------------------------------------------------------------
# Readings: as for 2-D maps.  A last block shorter than B is averaged over its in-bounds elements (the
# paper's shapes use floor(N/B), which only covers N divisible by B); a block longer than the row is the
# whole row; the block sum is the balanced pairwise tree over the B positions (neighbours first, positions
# outside the row count as +0.0).  The random stream, packing and blob are those of the 2-D form with the
# in-sample index e = c*N + i.
def lfc_mean_1d(x32: np.ndarray, block: int) -> np.ndarray:
    """H^L = AveragePooling1D(H), window = stride = B, for x32[M, C, N]; fp32 with the build's summation order."""
    x32 = np.asarray(x32, dtype=np.float32)
    m, c, n = x32.shape
    block = min(int(block), n)
    nb = -(-n // block)
    xp = np.zeros((m, c, nb * block), dtype=np.float32)
    xp[:, :, :n] = x32
    total = _pairwise_tree_sum(xp.reshape(m, c, nb, block), axis=-1)
    count = np.minimum(block, n - np.arange(nb) * block).astype(np.float32)
    return (total / count[None, None]).astype(np.float32)


def upsample_nearest_1d(lfc: np.ndarray, block: int, n: int) -> np.ndarray:
    """UpSampling1D(H^L): position i takes the value of block i // B."""
    return np.repeat(lfc, min(int(block), n), axis=2)[:, :, :n]


def compress_1d(x: np.ndarray, block: int, qbits: int, seed: int,
                x_dtype: str = F32, lfc_dtype: str = F32) -> Compressed:
    """Forward-loop steps of Algorithm 1 for a 1-D activation map H of shape Minibatch x Channel x N."""
    if qbits not in SUPPORTED_QBITS:
        raise ValueError("Q must divide 32")
    x32 = widen_input(x, x_dtype)
    m, c, n = x32.shape
    lfc = round_to_dtype(lfc_mean_1d(x32, block), lfc_dtype)
    r = (x32 - upsample_nearest_1d(lfc, block, n)).reshape(m, c * n)
    codes = np.empty((m, c * n), dtype=np.uint8)
    delta = np.empty(m, dtype=np.float32)
    step = np.empty(m, dtype=np.float32)
    e = np.arange(c * n, dtype=np.uint64)
    for i in range(m):
        delta[i], step[i], scale = sample_stats(r[i], qbits)
        codes[i] = quantize(r[i], delta[i], scale, divrng_fields(seed, i, e), qbits)
    words = pack_codes(codes.reshape(-1), qbits)
    layout = compressed_layout(m, c, 1, n, min(int(block), n), qbits, x_dtype, lfc_dtype)
    return Compressed((m, c, 1, n), min(int(block), n), qbits, x_dtype, lfc_dtype, lfc[:, :, None, :], codes, words,
                      delta, step, layout)


def decompress_1d(comp: Compressed) -> np.ndarray:
    """Backward-loop steps of Algorithm 1 for a 1-D map; returns fp32 values [M, C, N] rounded to the activation dtype."""
    m, c, _, n = comp.shape
    codes = unpack_codes(comp.words, comp.qbits, m * c * n).reshape(m, c * n)
    hh = np.empty((m, c * n), dtype=np.float32)
    for i in range(m):
        hh[i] = dequantize(codes[i], comp.delta[i], comp.step[i])
    xhat = upsample_nearest_1d(comp.lfc[:, :, 0, :], comp.block, n) + hh.reshape(m, c, n)
    return round_to_dtype(xhat.astype(np.float32), comp.x_dtype)


# ----------------------------------------------------------------------------------------
# 3-D activation maps  (appendix "Compression of 1D and 3D Activation Maps": Minibatch x Channel x N x N x N,
# average pooling and nearest up-sampling over B x B x B blocks, Quant and its inverse unchanged)
# ----------------------------------------------------------------------------------------
# Readings as for 2-D maps: ceil grid on every axis, a partial block is averaged over its in-bounds elements, a
# block larger than all three sides behaves like a block equal to the largest side; the block sum is the balanced
# pairwise tree along the depth axis first, then down the rows, then across the columns (positions outside the map
# count as +0.0; for depth 1 this is the 2-D order).  In-sample index e = ((c*D + d)*H + h)*W + w; random stream,
# packing and blob as before, with N*C*ceil(D/B)*ceil(H/B)*ceil(W/B) low-frequency values.
def _block3(d: int, h: int, w: int, block: int) -> int:
    return min(int(block), max(d, h, w))


def lfc_mean_3d(x32: np.ndarray, block: int) -> np.ndarray:
    """H^L = AveragePooling3D(H), window = stride = B, for x32[M, C, D, H, W]; fp32, the build's summation order."""
    x32 = np.asarray(x32, dtype=np.float32)
    m, c, d, h, w = x32.shape
    b = _block3(d, h, w, block)
    db, hb, wb = -(-d // b), -(-h // b), -(-w // b)
    xp = np.zeros((m, c, db * b, hb * b, wb * b), dtype=np.float32)
    xp[:, :, :d, :h, :w] = x32
    t = xp.reshape(m, c, db, b, hb, b, wb, b).transpose(0, 1, 2, 4, 6, 3, 5, 7)      # [..., depth, row, col] per block
    s = _pairwise_tree_sum(t, axis=-3)          # along the depth of every (row, col) position
    s = _pairwise_tree_sum(s, axis=-2)          # down the rows
    s = _pairwise_tree_sum(s, axis=-1)          # across the columns
    nd = np.minimum(b, d - np.arange(db) * b)
    nh = np.minimum(b, h - np.arange(hb) * b)
    nw = np.minimum(b, w - np.arange(wb) * b)
    count = (nd[:, None, None] * nh[None, :, None] * nw[None, None, :]).astype(np.float32)
    return (s / count[None, None]).astype(np.float32)


def upsample_nearest_3d(lfc: np.ndarray, block: int, d: int, h: int, w: int) -> np.ndarray:
    b = _block3(d, h, w, block)
    up = np.repeat(np.repeat(np.repeat(lfc, b, axis=2), b, axis=3), b, axis=4)
    return up[:, :, :d, :h, :w]


@dataclass
class Compressed3D:
    shape: tuple           # (M, C, D, H, W)
    block: int
    qbits: int
    x_dtype: str
    lfc_dtype: str
    lfc: np.ndarray        # [M, C, Db, Hb, Wb] fp32 values as stored
    codes: np.ndarray      # [M, C*D*H*W]
    words: np.ndarray
    delta: np.ndarray
    step: np.ndarray
    layout: Layout

    def blob(self) -> np.ndarray:
        out = np.zeros(self.layout.total_bytes, dtype=np.uint8)
        raw = self.lfc.astype("<f4").tobytes() if self.lfc_dtype == F32 else f32_to_bf16_bits(self.lfc).astype("<u2").tobytes()
        lo = self.layout
        out[lo.lfc_off:lo.lfc_off + lo.lfc_bytes] = np.frombuffer(raw, dtype=np.uint8)
        out[lo.packed_off:lo.packed_off + lo.packed_bytes] = np.frombuffer(self.words.astype("<u4").tobytes(), dtype=np.uint8)
        stats = np.stack([self.delta, self.step], axis=1).astype("<f4")
        out[lo.stats_off:lo.stats_off + lo.stats_bytes] = np.frombuffer(stats.tobytes(), dtype=np.uint8)
        return out


def layout_3d(m: int, c: int, d: int, h: int, w: int, block: int, qbits: int,
              x_dtype: str = F32, lfc_dtype: str = F32) -> Layout:
    b = _block3(d, h, w, block)
    tiles = m * c * (-(-d // b)) * (-(-h // b)) * (-(-w // b))
    lfc_bytes = tiles * _DTYPE_BYTES[lfc_dtype]
    packed_bytes = -(-(m * c * d * h * w * qbits) // 32) * 4
    packed_off = _align(lfc_bytes, SECTION_ALIGN)
    stats_off = _align(packed_off + packed_bytes, SECTION_ALIGN)
    return Layout(0, lfc_bytes, packed_off, packed_bytes, stats_off, 8 * m, stats_off + 8 * m,
                  lfc_bytes + packed_bytes + 8 * m, m * c * d * h * w * _DTYPE_BYTES[x_dtype])


def compress_3d(x: np.ndarray, block: int, qbits: int, seed: int,
                x_dtype: str = F32, lfc_dtype: str = F32) -> Compressed3D:
    """Forward-loop steps of Algorithm 1 for a 3-D activation map H of shape Minibatch x Channel x D x H x W."""
    if qbits not in SUPPORTED_QBITS:
        raise ValueError("Q must divide 32")
    x32 = widen_input(x, x_dtype)
    m, c, d, h, w = x32.shape
    per = c * d * h * w
    lfc = round_to_dtype(lfc_mean_3d(x32, block), lfc_dtype)
    r = (x32 - upsample_nearest_3d(lfc, block, d, h, w)).reshape(m, per)
    codes = np.empty((m, per), dtype=np.uint8)
    delta = np.empty(m, dtype=np.float32)
    step = np.empty(m, dtype=np.float32)
    e = np.arange(per, dtype=np.uint64)
    for i in range(m):
        delta[i], step[i], scale = sample_stats(r[i], qbits)
        codes[i] = quantize(r[i], delta[i], scale, divrng_fields(seed, i, e), qbits)
    words = pack_codes(codes.reshape(-1), qbits)
    return Compressed3D((m, c, d, h, w), _block3(d, h, w, block), qbits, x_dtype, lfc_dtype, lfc, codes, words, delta, step,
                        layout_3d(m, c, d, h, w, block, qbits, x_dtype, lfc_dtype))


def decompress_3d(comp: Compressed3D) -> np.ndarray:
    m, c, d, h, w = comp.shape
    per = c * d * h * w
    codes = unpack_codes(comp.words, comp.qbits, m * per).reshape(m, per)
    hh = np.empty((m, per), dtype=np.float32)
    for i in range(m):
        hh[i] = dequantize(codes[i], comp.delta[i], comp.step[i])
    xhat = upsample_nearest_3d(comp.lfc, comp.block, d, h, w) + hh.reshape(m, c, d, h, w)
    return round_to_dtype(xhat.astype(np.float32), comp.x_dtype)
