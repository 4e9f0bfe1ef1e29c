"""TEST INFRASTRUCTURE. What it would cost in accuracy to hand all-BASE tiles of an fp16 pool to
8-bit tensor-core instructions without expanding them (Sec. 4.1 / Tab. 1: an fp16 cache whose BASE
state is the high byte, i.e. an E5M2 number; App. C.5 compares with a static FP8 cache).

Reading (named "FP8 operands"): for a KV tile of 128 tokens whose pages are all BASE,
  - K and V enter as the E5M2 numbers they already are (no rounding at all);
  - the query row is rounded to an 8-bit float (E4M3 or E5M2, round to nearest even, saturating),
  - the probabilities of that tile are rounded to an 8-bit float after a scaling by 2^8 that keeps
    them inside the E4M3 range, and unscaled after the product;
every other tile (mixed or TARGET) is taken in 16 bits as usual. Sums in float64: the only
differences to the plain oracle are the two 8-bit roundings. Written from the format definitions
(E4M3: bias 7, 3 mantissa bits, no infinities, largest finite 448; E5M2: bias 15, 2 mantissa
bits), pinned in tests/test_oracle_fp8_reading.py by brute force over all 256 codes."""
import numpy as np


def _decode_table(exp_bits, man_bits, bias, fn_variant):
    """All non-negative finite values of an 8-bit float format, from its definition."""
    vals = []
    for code in range(128):
        e = code >> man_bits
        m = code & ((1 << man_bits) - 1)
        if fn_variant:                                    # E4M3: only exponent 15, mantissa 7 is NaN
            if e == (1 << exp_bits) - 1 and m == (1 << man_bits) - 1:
                continue
        elif e == (1 << exp_bits) - 1:                    # E5M2: infinities and NaNs
            continue
        vals.append(m * 2.0 ** (1 - bias - man_bits) if e == 0 else (1 + m / (1 << man_bits)) * 2.0 ** (e - bias))
    return np.array(sorted(set(vals)))


E4M3_VALUES = _decode_table(4, 3, 7, True)
E5M2_VALUES = _decode_table(5, 2, 15, False)


def round_to_format(x, man_bits, min_exp, max_finite):
    """Round to nearest even in a binary float format with `man_bits` stored mantissa bits, smallest
    normal exponent `min_exp` (gradual underflow below it) and saturation at +-max_finite."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -60)))
    e = np.maximum(e, min_exp)
    q = 2.0 ** (e - man_bits)                             # spacing of the format at |x|
    r = np.rint(a / q) * q                                # numpy rounds halves to even
    return np.sign(x) * np.minimum(r, max_finite)


def e4m3(x):
    return round_to_format(x, 3, -6, 448.0)


def e5m2(x):
    return round_to_format(x, 2, -14, 57344.0)


def attention_row(q, k, v, sm_scale, tile_is_base=None, q_round=None, p_round=None, tile=128):
    """One query row against L tokens (k, v float64 [L][D], already dequantised). Tiles listed in
    tile_is_base take the 8-bit reading: scores from the rounded query, probabilities rounded
    (after the 2^8 scaling) before they multiply V and before they are summed."""
    L = k.shape[0]
    n_tiles = -(-L // tile)
    if tile_is_base is None:
        tile_is_base = np.zeros(n_tiles, bool)
    s = np.empty(L)
    q8 = q_round(q) if q_round is not None else q
    for t in range(n_tiles):
        sl = slice(t * tile, min(L, (t + 1) * tile))
        s[sl] = (k[sl] @ (q8 if tile_is_base[t] else q)) * sm_scale
    p = np.exp(s - s.max())
    if p_round is not None:
        for t in range(n_tiles):
            if tile_is_base[t]:
                sl = slice(t * tile, min(L, (t + 1) * tile))
                p[sl] = p_round(p[sl] * 256.0) / 256.0
    return (p @ v) / p.sum()
