"""Pins for the oracle's integer AbsMax quantiser (Eq. 4), CPU only."""
import os

import numpy as np

from oracle import tweo_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_qmax_values_from_eq4():
    consts = {l.split()[0]: l.split()[1] for l in open(os.path.join(GOLD, "paper_constants.txt"))
              if l.strip() and l[0] != "#"}
    assert orc.absmax_qmax(8) == int(consts["Q_8"]) == 127
    assert orc.absmax_qmax(6) == int(consts["Q_6"]) == 31
    assert orc.absmax_qmax(4) == 7


def test_absmax_properties():
    g = np.random.Generator(np.random.PCG64(41))
    x = g.standard_normal(1000) * 3
    for bits in (8, 6):
        Q = orc.absmax_qmax(bits)
        s = orc.absmax_scale(x, 1e-6)
        assert s == np.max(np.abs(x)) + 1e-6
        q = orc.absmax_quantize(x, bits, s)
        assert q.max() <= Q and q.min() >= -Q
        assert abs(q[np.argmax(np.abs(x))]) == Q            # the largest element maps to +-Q_b
        assert np.array_equal(q, np.rint(x / s * Q).astype(np.int32))   # numpy rint = ties-to-even
        deq = orc.absmax_dequantize(q, bits, s)
        assert np.max(np.abs(deq - x)) <= s / Q / 2 * (1 + 1e-12)
        assert np.array_equal(orc.absmax_quantize(deq, bits, s), q)   # idempotent
    # ties to even, and clamping under a static (too small) scale
    assert list(orc.absmax_quantize(np.array([0.5, 1.5, 2.5, -0.5, 300.0, -300.0]), 8, 127.0)) == [0, 2, 2, 0, 127, -127]
