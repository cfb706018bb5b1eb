"""Pins of the oracle's fp8 chunk codec (compressed KV store) against things other than itself: the
library's float8_e4m3fn type, hand-computed codes, closed-form bounds and round trips."""
import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle
from _util import rand_bits


def _torch_decode(codes):
    return torch.from_numpy(np.asarray(codes, dtype=np.uint8)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def test_code_values_match_the_library_type():
    codes = [c for c in range(256) if c & 0x7f != 0x7f]          # 0x7f / 0xff are the NaN codes
    mine = np.array([oracle.e4m3_value(c) for c in codes])
    assert np.array_equal(mine, _torch_decode(codes))
    assert mine.max() == 448.0 and np.min(np.abs(mine[mine != 0])) == 2.0 ** -9


def test_hand_computed_codes():
    # sign | exponent (bias 7) | mantissa
    for x, code in [(1.0, 0x38), (-1.0, 0xb8), (448.0, 0x7e), (2.0 ** -9, 0x01), (0.5, 0x30), (1.5, 0x3c), (240.0, 0x77),
                    (2.0 ** -6, 0x08), (7 * 2.0 ** -9, 0x07), (0.0, 0x00), (-0.0, 0x00)]:
        assert oracle.e4m3_encode(x) == code, (x, hex(oracle.e4m3_encode(x)))
    # ties go to the even mantissa: 1.0625 lies between 1.0 (0x38) and 1.125 (0x39); 1.1875 between 0x39 and 1.25 (0x3a)
    assert oracle.e4m3_encode(1.0625) == 0x38 and oracle.e4m3_encode(1.1875) == 0x3a
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00 and oracle.e4m3_encode(3 * 2.0 ** -10) == 0x02   # subnormal ties
    assert oracle.e4m3_encode(1000.0) == 0x7e and oracle.e4m3_encode(-1000.0) == 0xfe               # saturation


def test_encode_inverts_value_and_is_monotonic():
    for c in range(1, 0x7f):
        assert oracle.e4m3_encode(oracle.e4m3_value(c)) == c
        assert oracle.e4m3_encode(-oracle.e4m3_value(c)) == (c | 0x80)
    xs = np.linspace(-460, 460, 20001)
    vals = np.array([oracle.e4m3_value(oracle.e4m3_encode(x)) for x in xs])
    assert np.all(np.diff(vals) >= 0)


def test_encode_matches_the_library_cast_on_random_values():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.uniform(-448, 448, 20000), rng.normal(0, 1, 20000), rng.uniform(-0.02, 0.02, 20000)]).astype(np.float32)
    lib = x.copy()
    lib_codes = torch.from_numpy(lib).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = np.array([oracle.e4m3_encode(float(v)) for v in x], dtype=np.uint8)
    same = mine == lib_codes
    zero = (mine & 0x7f) == 0                                      # the oracle stores no negative zero
    assert np.all(same | (zero & ((lib_codes & 0x7f) == 0)))


def test_block_exponent_closed_forms():
    # smallest e with amax * 2^-e <= 448 = 1.75 * 2^8
    for amax, e in [(448.0, 0), (450.0, 1), (896.0, 1), (900.0, 2), (1.0, -8), (1.75, -8), (1.7578125, -7), (224.0, -1),
                    (3.5, -7), (0.0, 0), (2.0 ** -140, -127), (2.0 ** 127, 119)]:
        assert oracle.fp8_block_exponent(amax) == e, (amax, oracle.fp8_block_exponent(amax))
        if amax > 0 and -127 < e:
            assert amax * 2.0 ** -e <= 448 < amax * 2.0 ** -(e - 1)


@pytest.mark.parametrize("n,shift", [(1, 0), (63, 0), (64, 3), (65, -5), (200, 0)])
def test_blob_round_trip_bounds_and_bf16_exactness(n, shift):
    sh = oracle.Shape(2, 4, 2, 64)
    blob = rand_bits(31, n, (2, 2, 2, n, 64), shift)
    blob[0, 1, 1, : min(n, 64)] = 0                                 # an all-zero block
    codes, exps = oracle.fp8_quantize_blob(sh, blob)
    deq = oracle.fp8_dequantize_blob(sh, codes, exps)
    x, y = mi.bf16_bits_to_f64(blob), mi.bf16_bits_to_f64(deq)
    # what the codes stand for, computed here from the definition
    e_full = np.repeat(exps.astype(np.float64), 64, axis=3)[:, :, :, :n, None]
    y_def = _torch_decode(codes.reshape(-1)).reshape(codes.shape) * 2.0 ** e_full
    assert np.array_equal(y, y_def)                                 # value(code) * 2^e is a bf16 number: nothing was rounded
    # error bound: half an e4m3 step of the scaled value (relative 2^-4 for normals, absolute 2^-10 for subnormals)
    assert np.all(np.abs(x - y) <= np.maximum(np.abs(x) * 2.0 ** -4, 2.0 ** (e_full - 10.0)) * (1 + 1e-12))
    assert np.all(exps[0, 1, 1, 0] == 0) and np.all(codes[0, 1, 1, : min(n, 64)] == 0)
    # the block maximum uses the top binade of the code range: scaled amax in (224, 448]
    xb = np.abs(x[1, 0, 0, : min(n, 64)]).max()
    assert 224 < xb * 2.0 ** -float(exps[1, 0, 0, 0]) <= 448
    # quantising what a compressed chunk stands for gives the same codes back
    codes2, exps2 = oracle.fp8_quantize_blob(sh, deq)
    assert np.array_equal(mi.bf16_bits_to_f64(oracle.fp8_dequantize_blob(sh, codes2, exps2)), y)
