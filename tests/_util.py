"""Shared helpers of the GPU parity tests (comparison against the CPU oracle)."""
import numpy as np

import matkv_inputs as mi

# tolerances: max-abs and mean-abs are the target stated for unit-scale bf16 data; the relative RMS
# and lse bounds are added because |o| shrinks like sqrt(e/n) at long context (an all-zero output
# would pass an absolute 1e-2 there).  bf16 output rounding alone gives 2^-9 relative per element.
MAX_ABS, MEAN_ABS, REL_RMS, LSE_ABS = 1e-2, 1e-3, 1e-2, 1e-3


def rand_bits(seed, stream, shape, shift=0):
    return mi.normal_bf16(seed, stream, int(np.prod(shape)), shift).reshape(shape)


def check(o_bits, o_ref, lse, lse_ref, what=""):
    o = mi.bf16_bits_to_f64(np.asarray(o_bits)).reshape(o_ref.shape)
    err = np.abs(o - o_ref)
    assert np.all(np.isfinite(o)), f"{what}: non-finite output"
    mx, mean = float(err.max()), float(err.mean())
    rel = float(np.linalg.norm(o - o_ref) / max(np.linalg.norm(o_ref), 1e-30))
    assert mx <= MAX_ABS, f"{what}: max-abs {mx}"
    assert mean <= MEAN_ABS, f"{what}: mean-abs {mean}"
    assert rel <= REL_RMS, f"{what}: relative rms {rel}"
    if lse is not None:
        le = float(np.max(np.abs(np.asarray(lse, dtype=np.float64).reshape(lse_ref.shape) - lse_ref)))
        assert le <= LSE_ABS, f"{what}: lse abs {le}"
    return mx, mean, rel
