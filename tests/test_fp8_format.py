"""Host-side check of the tests' own E4M3 quantiser (tests/_fp8.py) against the oracle's rounding routine, and of the
table against the format's landmarks.  No GPU."""
import numpy as np

import oracle
from _fp8 import e4m3_table, quantize_e4m3


def test_host_quantiser_agrees_with_the_oracle_routine():
    rng = np.random.default_rng(5)
    xs = np.concatenate([rng.normal(size=400) * 3, [0.0, 448.0, 500.0, -1000.0, 2.0 ** -9, 2.0 ** -10, 1.0625, 1.1875, 0.0009765625 * 1.5]])
    tab = e4m3_table()
    for x in xs.astype(np.float32):
        assert tab[quantize_e4m3(np.float64(x))] == oracle.round_fp8(float(x), "e4m3"), x


def test_table_landmarks():
    tab = e4m3_table()
    assert tab[0x38] == 1.0 and tab[0x7E] == 448.0 and tab[0x01] == 2.0 ** -9 and tab[0x08] == 2.0 ** -6
    assert np.isnan(tab[0x7F]) and np.isnan(tab[0xFF]) and tab[0xB8] == -1.0
    assert np.all(np.diff(tab[:0x7F]) > 0)                       # the non-negative codes are ordered
    assert quantize_e4m3(np.float64(-1e-6)) == 0x80 and quantize_e4m3(np.float64(1e9)) == 0x7E
