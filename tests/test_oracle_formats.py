"""Pins for the oracle's number formats, table fold and quantiser (CPU only).

Each check ties the oracle to something other than itself: a library conversion routine
(numpy's float16), exact rational arithmetic, or an invariant the documented format fixes.
"""
import os
from fractions import Fraction

import numpy as np
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _bf16_val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def test_lut_fold_exhaustive(oracle):
    rows = [tuple(map(int, l.split())) for l in open(os.path.join(GOLD, "lut_fold.txt")) if l[0] != "#"]
    assert len(rows) == 9
    for a0, fl, a in rows:
        assert oracle.lut_fold(a0, fl) == a


def test_f16_rne_matches_numpy_on_stratified_floats(oracle):
    # every exponent that matters for fp16 (2^-27 .. 2^16) x a spread of mantissas, both signs,
    # plus exact ties and their neighbours; compared with numpy's own fp32 -> fp16 conversion
    rng = np.random.default_rng(7)
    exps = np.arange(127 - 27, 127 + 16, dtype=np.uint32)
    man = np.concatenate([rng.integers(0, 1 << 23, 4000, dtype=np.uint32),
                          np.array([0, 1, 0x1000, 0x0FFF, 0x1001, 0x3000, 0x2FFF, 0x3001, 0x7FFFFF, 0x7FF000,
                                    0x7FEFFF, 0x7FF001, 0x400000, 0x200000, 0x600000], dtype=np.uint32)])
    bits = (exps[:, None] << 23 | man[None, :]).reshape(-1)
    bits = np.concatenate([bits, bits | np.uint32(0x80000000)])
    x = bits.view(np.float32)
    want = x.astype(np.float16).view(np.uint16)
    fin = np.isfinite(x.astype(np.float16))
    L = oracle.lib()
    got = np.fromiter((L.orc_f32_to_f16_rne(float(v)) for v in x), dtype=np.uint16, count=x.size)
    assert np.array_equal(got[fin], want[fin])
    # where IEEE conversion overflows to infinity the documented reading saturates at 65504
    assert np.all((got[~fin] & 0x7FFF) == 0x7BFF)


def test_f16_decode_matches_numpy_for_all_patterns(oracle):
    L = oracle.lib()
    h = np.arange(0, 1 << 16, dtype=np.uint16)
    want = h.view(np.float16).astype(np.float32)
    got = np.fromiter((L.orc_f16_to_f32(int(v)) for v in h), dtype=np.float32, count=h.size)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_f16_special_cases(oracle):
    assert oracle.f32_to_f16_bits(0.0) == 0
    assert oracle.f32_to_f16_bits(65504.0) == 0x7BFF
    assert oracle.f32_to_f16_bits(65520.0) == 0x7BFF      # would round to inf: saturates
    assert oracle.f32_to_f16_bits(1e30) == 0x7BFF
    assert oracle.f32_to_f16_bits(2.0 ** -24) == 1        # smallest subnormal
    assert oracle.f32_to_f16_bits(2.0 ** -25) == 0        # exact tie to even -> 0
    assert oracle.f32_to_f16_bits(np.nextafter(np.float32(2.0 ** -25), np.float32(1))) == 1
    assert oracle.f32_to_f16_bits(1.0 + 2.0 ** -11) == 0x3C00   # tie -> even
    assert oracle.f32_to_f16_bits(1.0 + 3 * 2.0 ** -11) == 0x3C02


def _groups(seed, n, scale=1.0):
    rng = np.random.default_rng(seed)
    return _bf16_bits((rng.standard_normal((n, 32)) * scale).astype(np.float32))


def test_quantizer_invariants_on_random_groups(oracle):
    for scale in (1.0, 1e-3, 1e3):
        for xb in _groups(11, 3000, scale):
            x = _bf16_val(xb).astype(np.float64)
            sb, codes = oracle.quantize_group(xb)
            s = float(np.array([sb], np.uint16).view(np.float16)[0])
            assert codes.min() >= 1 and codes.max() <= 15
            amax = np.abs(x).max()
            # the scale is fp16(amax / 7) computed in fp32
            assert sb == int(np.float16(np.float32(amax) / np.float32(7.0)).view(np.uint16))
            i = int(np.abs(x).argmax())
            assert int(codes[i]) - 8 == (7 if x[i] > 0 else -7)
            xh = (codes.astype(np.int64) - 8) * s
            assert np.all(np.abs(x - xh) <= 0.5 * s * (1 + 2.0 ** -10) + 1e-30)


def test_quantizer_codes_are_nearest_integers_in_exact_arithmetic(oracle):
    # brute force with rationals: the code must be a nearest integer to x / s (either neighbour is
    # accepted only when x / s is within 2^-20 of a tie, where the fp32 recipe may round either way)
    for xb in _groups(5, 400):
        sb, codes = oracle.quantize_group(xb)
        s = Fraction(float(np.array([sb], np.uint16).view(np.float16)[0]))
        for xi, c in zip(_bf16_val(xb), codes):
            r = Fraction(float(xi)) / s
            r = max(Fraction(-7), min(Fraction(7), r))
            assert abs(r - (int(c) - 8)) <= Fraction(1, 2) + Fraction(1, 1 << 20)


def test_quantizer_degenerate_groups(oracle):
    sb, codes = oracle.quantize_group(np.zeros(32, np.uint16))
    assert sb == 0 and np.all(codes == 8)
    # negative zeros are still zeros
    sb, codes = oracle.quantize_group(np.full(32, 0x8000, np.uint16))
    assert sb == 0 and np.all(codes == 8)
    # a constant group maps every element to +-7
    xb = _bf16_bits(np.full(32, 1.75, np.float32))
    sb, codes = oracle.quantize_group(xb)
    assert np.all(codes == 15) and sb == int(np.float16(0.25).view(np.uint16))
    xb = _bf16_bits(np.full(32, -3.0, np.float32))
    _, codes = oracle.quantize_group(xb)
    assert np.all(codes == 1)
    # values so small that the fp16 scale underflows to zero: all codes 8
    xb = _bf16_bits(np.full(32, 1e-9, np.float32))
    sb, codes = oracle.quantize_group(xb)
    assert sb == 0 and np.all(codes == 8)
    # values so large that amax / 7 exceeds fp16: the scale saturates, codes clamp to +-7
    xb = _bf16_bits(np.array([1e6, -1e6] * 16, np.float32))
    sb, codes = oracle.quantize_group(xb)
    assert sb == 0x7BFF and set(codes.tolist()) == {1, 15}
    # subnormal fp16 scale is kept (no flush to zero)
    xb = _bf16_bits(np.linspace(-1, 1, 32).astype(np.float32) * 1e-5)
    sb, codes = oracle.quantize_group(xb)
    assert 0 < sb < 0x0400 and codes.min() == 1 and codes.max() == 15


def test_quantizer_sign_symmetry(oracle):
    for xb in _groups(3, 500):
        sb, codes = oracle.quantize_group(xb)
        sb2, codes2 = oracle.quantize_group(xb ^ np.uint16(0x8000))
        assert sb == sb2
        assert np.array_equal(codes2.astype(np.int64) - 8, -(codes.astype(np.int64) - 8))


def test_action_cost_table_matches_formats():
    for line in open(os.path.join(GOLD, "action_cost.txt")):
        if line[0] == "#":
            continue
        n_kv, r, l, h = map(int, line.split())
        assert r == 0
        assert h == 2 * n_kv * 128 * 2                      # K and V, bf16
        assert l == 2 * n_kv * (128 // 2 + (128 // 32) * 2)  # nibbles + one fp16 scale per 32 values
        assert 0 < l < h and abs(l / h - 0.28125) < 1e-12


# ---- the 8-bit variant of RETAIN-LOW (policy low_bits = 8): same recipe with 127 in place of 7

def test_quantizer8_invariants_and_exact_nearest(oracle):
    for scale in (1.0, 1e-3, 1e3):
        for xb in _groups(21, 1500, scale):
            x = _bf16_val(xb).astype(np.float64)
            sb, codes = oracle.quantize_group(xb, bits=8)
            s = float(np.array([sb], np.uint16).view(np.float16)[0])
            assert codes.min() >= 1 and codes.max() <= 255
            assert sb == int(np.float16(np.float32(np.abs(x).max()) / np.float32(127.0)).view(np.uint16))
            xh = (codes.astype(np.int64) - 128) * s
            assert np.all(np.abs(x - xh) <= 0.5 * s * (1 + 2.0 ** -9) + 1e-30)
    for xb in _groups(22, 300):
        sb, codes = oracle.quantize_group(xb, bits=8)
        s = Fraction(float(np.array([sb], np.uint16).view(np.float16)[0]))
        for xi, c in zip(_bf16_val(xb), codes):
            r = max(Fraction(-127), min(Fraction(127), Fraction(float(xi)) / s))
            assert abs(r - (int(c) - 128)) <= Fraction(1, 2) + Fraction(1, 1 << 16)


def test_quantizer8_degenerate_groups_and_symmetry(oracle):
    sb, codes = oracle.quantize_group(np.zeros(32, np.uint16), bits=8)
    assert sb == 0 and np.all(codes == 128)
    xb = _bf16_bits(np.full(32, 1e-9, np.float32))                  # scale underflows to zero
    sb, codes = oracle.quantize_group(xb, bits=8)
    assert sb == 0 and np.all(codes == 128)
    xb = _bf16_bits(np.array([1e7, -1e7] * 16, np.float32))         # scale saturates, codes clamp
    sb, codes = oracle.quantize_group(xb, bits=8)
    assert sb == 0x7BFF and set(codes.tolist()) == {1, 255}
    xb = _bf16_bits(np.full(32, 127.0, np.float32))                 # scale exactly 1: codes are the values
    sb, codes = oracle.quantize_group(xb, bits=8)
    assert sb == 0x3C00 and np.all(codes == 255)
    xb = _bf16_bits(np.arange(-16, 16, dtype=np.float32) * 8 - 1)   # amax 129 -> not a clean scale; still symmetric
    for xb in _groups(23, 300):
        sb, codes = oracle.quantize_group(xb, bits=8)
        sb2, codes2 = oracle.quantize_group(xb ^ np.uint16(0x8000), bits=8)
        assert sb == sb2 and np.array_equal(codes2.astype(np.int64) - 128, -(codes.astype(np.int64) - 128))


# ---- the 2-bit variant (policy low_bits = 2): three levels -s, 0, +s with s = fp16(amax)

def test_quantizer2_is_the_nearest_of_three_levels(oracle):
    for scale in (1.0, 1e-3, 1e3):
        for xb in _groups(31, 600, scale):
            x = _bf16_val(xb).astype(np.float64)
            sb, codes = oracle.quantize_group(xb, bits=2)
            assert sb == int(np.float16(np.float32(np.abs(x).max())).view(np.uint16))      # amax / 1
            s = Fraction(float(np.array([sb], np.uint16).view(np.float16)[0]))
            assert set(codes.tolist()) <= {1, 2, 3}
            for xi, c in zip(x, codes):
                # brute force over the three levels in exact arithmetic; a value half-way goes to the even level 0
                d = [abs(Fraction(float(xi)) - lv * s) for lv in (-1, 0, 1)]
                best = min(d)
                picks = [lv for lv, di in zip((-1, 0, 1), d) if di - best <= s * Fraction(1, 1 << 16)]
                assert (int(c) - 2) in picks
                if len(picks) > 1 and abs(abs(Fraction(float(xi))) - s / 2) == 0:
                    assert int(c) == 2


def test_quantizer2_degenerate_groups_and_symmetry(oracle):
    sb, codes = oracle.quantize_group(np.zeros(32, np.uint16), bits=2)
    assert sb == 0 and np.all(codes == 2)
    xb = _bf16_bits(np.full(32, 1e-9, np.float32))                  # scale underflows to zero
    sb, codes = oracle.quantize_group(xb, bits=2)
    assert sb == 0 and np.all(codes == 2)
    xb = _bf16_bits(np.array([1e7, -1e7] * 16, np.float32))         # scale saturates, codes clamp
    sb, codes = oracle.quantize_group(xb, bits=2)
    assert sb == 0x7BFF and set(codes.tolist()) == {1, 3}
    xb = _bf16_bits(np.array([1.0, 0.5, 0.25, -0.5, -0.75, -1.0, 0.0, 0.51] * 4, np.float32))
    sb, codes = oracle.quantize_group(xb, bits=2)                   # ties at half the scale go to the even level 0
    assert sb == 0x3C00 and codes[:8].tolist() == [3, 2, 2, 2, 1, 1, 2, 3]
    for xb in _groups(32, 300):
        sb, codes = oracle.quantize_group(xb, bits=2)
        sb2, codes2 = oracle.quantize_group(xb ^ np.uint16(0x8000), bits=2)
        assert sb == sb2 and np.array_equal(codes2.astype(np.int64) - 2, -(codes.astype(np.int64) - 2))


def test_eight_bit_is_finer_than_four_bit(oracle):
    # the same group at both widths: the 8-bit reconstruction error is never larger than half a 4-bit step
    for xb in _groups(24, 300):
        x = _bf16_val(xb).astype(np.float64)
        s4, c4 = oracle.quantize_group(xb, bits=4)
        s8, c8 = oracle.quantize_group(xb, bits=8)
        f = lambda b: float(np.array([b], np.uint16).view(np.float16)[0])
        e4 = np.abs(x - (c4.astype(np.int64) - 8) * f(s4)).max()
        e8 = np.abs(x - (c8.astype(np.int64) - 128) * f(s8)).max()
        assert e8 <= e4 + 1e-12 and e8 <= 0.5 * f(s8) * (1 + 2.0 ** -9)
