"""The oracle against the hand-derived fixture in tests/golden/ (values fixed by the paper's equations)."""
import math
import os

import numpy as np

from oracle.kdkl_oracle import kdkl_oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _rows():
    with open(os.path.join(HERE, "golden", "two_entry_vocabulary.txt")) as f:
        return [[float(x) for x in line.split()] for line in f if line.strip() and not line.startswith("#")]


def test_fixture_is_what_the_equations_say():
    full, half = _rows()
    assert abs(full[1] - math.log(1.5)) < 1e-15 and abs(full[2] - math.log(3.0)) < 1e-15
    assert abs(half[1] - (0.5 * math.log(3.0) - math.log(2.0))) < 1e-15
    assert abs(full[5] + math.log(2.0) / 3) < 1e-15 and abs(half[5] + math.log(2.0) / 6) < 1e-15


def test_oracle_reproduces_hand_derived_case():
    h = np.array([[1.0]])
    W = np.array([[math.log(2.0)], [0.0]])
    idx = np.array([[0]], dtype=np.int32)
    val = np.array([[0.7]])                       # any value: K = 1, so only the normaliser matters
    for mass, loss, logz, dz0, dz1, dH, dW0, dW1 in _rows():
        lse = None if mass == 1.0 else np.array([0.7 - math.log(mass)])
        o = kdkl_oracle(h, W, idx, val, teacher_lse=lse)
        assert abs(o["M"][0] - mass) < 1e-15
        assert abs(o["loss"] - loss) < 1e-14 and abs(o["logZ"][0] - logz) < 1e-14
        assert abs(o["dH"][0, 0] - dH) < 1e-14
        np.testing.assert_allclose(o["dW"][:, 0], [dW0, dW1], rtol=0, atol=1e-14)
        assert abs(o["gathered_logits"][0, 0] - math.log(2.0)) < 1e-15
