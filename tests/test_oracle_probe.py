"""Pins for the oracle's distortion probe (the inner term of Eq. 4). CPU only."""
import numpy as np


def test_closed_forms(oracle):
    rng = np.random.default_rng(5)
    a = rng.standard_normal((6, 8, 128)).astype(np.float32)
    per, tot = oracle.distortion(a, a)
    assert np.all(per == 0) and tot == 0                         # identical outputs: no distortion
    b = a.copy()
    b[2, 3, :] += np.float32(0.5)                                # one head off by 0.5 in every dim: 128 * 0.25
    b[2, 5, 7] += np.float32(2.0)                                # another head off in one dim: 4 < 32
    b[4, 0, 0] -= np.float32(3.0)                                # 9
    per, tot = oracle.distortion(a, b)
    want = np.zeros(6)
    want[2] = ((a[2, 3].astype(np.float64) - b[2, 3].astype(np.float64)) ** 2).sum()
    want[4] = (float(a[4, 0, 0]) - float(b[4, 0, 0])) ** 2
    assert abs(want[2] - 32.0) < 1e-4 and abs(want[4] - 9.0) < 1e-5
    assert np.allclose(per, want, rtol=0, atol=1e-12) and abs(tot - want.sum()) < 1e-12


def test_against_numpy_and_symmetry(oracle):
    rng = np.random.default_rng(6)
    a = rng.standard_normal((40, 32, 128)).astype(np.float32)
    b = (a + 0.01 * rng.standard_normal(a.shape)).astype(np.float32)
    per, tot = oracle.distortion(a, b)
    ref = ((a.astype(np.float64) - b.astype(np.float64)) ** 2).sum(-1).max(-1)
    assert np.allclose(per, ref, rtol=1e-13, atol=0) and abs(tot - ref.sum()) < 1e-9
    per2, _ = oracle.distortion(b, a)
    assert np.array_equal(per, per2)
