"""The 8-byte intermediate-buffer entry (lt_format 2) restated in numpy for the tests.

Four 16-bit words per hit.  Word ch (0..2) is 4096 * (alpha dC/dalpha)_ch (clamped to +-60000) rounded to nine
mantissa bits (nearest, ties to even) and stored as an IEEE half, whose lowest bit -- zero after that rounding in
the normal range -- is replaced by the flag "colour channel ch is not clamped"; word 3 is the half nearest to
4096 * w.  A decoded colour word is therefore within
2^-10 (relative) of the encoder's input while that input times 4096 stays in the half's normal range, and w within
2^-11.
"""
import numpy as np

SCALE = 4096.0
LIMIT = 60000.0
REL_X = 2.0 ** -10
REL_W = 2.0 ** -11
TINY = 2.0 ** -14 / SCALE      # below this the half is subnormal: absolute error up to 2^-25 / SCALE ... 2^-24 / SCALE
ABS_SUB = 2.0 ** -23 / SCALE   # bound on the absolute error of a colour word in the subnormal range


def encode(entry, flags):
    """entry [H,4] float, flags [H] uint8 -> [H,4] uint16."""
    entry = np.asarray(entry, dtype=np.float64)
    y = np.clip(entry * SCALE, -LIMIT, LIMIT)
    m, e = np.frexp(y[:, :3])                              # |m| in [0.5, 1): nine mantissa bits = multiples of 2^-10
    y9 = np.ldexp(np.round(m * 1024.0) / 1024.0, e)        # np.round: ties to even
    c = y9.astype(np.float16).view(np.uint16).astype(np.uint32)
    b = y.astype(np.float16).view(np.uint16).astype(np.uint32)
    f = np.asarray(flags, dtype=np.uint32)[:, None] >> np.arange(3, dtype=np.uint32)[None, :] & 1
    out = np.empty(b.shape, dtype=np.uint16)
    out[:, :3] = ((c & 0xFFFE) | f).astype(np.uint16)
    out[:, 3] = b[:, 3].astype(np.uint16)
    return out


def decode(words):
    """[H,4] uint16 -> (entry [H,4] float64, flags [H] uint8)."""
    words = np.ascontiguousarray(words, dtype=np.uint16)
    flags = ((words[:, 0] & 1) | ((words[:, 1] & 1) << 1) | ((words[:, 2] & 1) << 2)).astype(np.uint8)
    clean = words.copy()
    clean[:, :3] &= 0xFFFE
    return clean.view(np.float16).astype(np.float64) / SCALE, flags
