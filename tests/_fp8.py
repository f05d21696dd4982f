"""The E4M3 format by its definition, for tests: the table of its 256 values and a brute-force quantiser."""
import numpy as np


def e4m3_table():
    """The 256 values of the E4M3 format by its definition (bias 7, subnormals, no infinity, S.1111.111 = NaN)."""
    t = np.empty(256, np.float64)
    for b in range(256):
        s, e, m = b >> 7, (b >> 3) & 15, b & 7
        v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[b] = np.nan if (e == 15 and m == 7) else (-v if s else v)
    return t


def quantize_e4m3(x):
    """Nearest E4M3 value of |x| (ties to the even code, saturating at 448) with the sign of x: brute force over the
    table of the non-negative codes."""
    tab = e4m3_table()
    codes = np.arange(0x7F)                                            # 0 .. 0x7E: the finite non-negative values
    vals = tab[codes]
    x = np.asarray(x, np.float64)
    mag = np.minimum(np.abs(x), 448.0)
    dist = np.abs(mag[..., None] - vals)
    best = dist.min(-1, keepdims=True)
    cand = np.where(dist == best, codes, 1 << 20)                      # all nearest codes (two on a tie)
    even = np.where((cand & 1) == 0, cand, 1 << 20)
    pick = np.where(even.min(-1) < (1 << 20), even.min(-1), cand.min(-1))
    return (pick | np.where(np.signbit(x), 0x80, 0)).astype(np.uint8)
