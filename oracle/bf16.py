"""Round-to-nearest-even conversion to the two 16-bit operand formats: bfloat16, written from the format's
definition (1 sign, 8 exponent, 7 mantissa bits = the upper half of an IEEE binary32), and IEEE binary16
(1 sign, 5 exponent, 10 mantissa bits), for which numpy's own conversion is the library step."""
import numpy as np


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Return `a` (any float dtype) rounded to the nearest bf16 value, ties to even, as fp64.

    The value is first rounded to binary32 (as the fp32 master copy of a mixed-precision
    level would hold it) and then to bf16.  Inf/NaN pass through."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32)
    finite = np.isfinite(f)
    out = np.where(finite, out, f)
    return out.astype(np.float64).reshape(np.shape(a))


FP16_MAX = 65504.0          # largest finite binary16 value; magnitudes from 65520 up round to infinity


def round_to_fp16(a: np.ndarray) -> np.ndarray:
    """Return `a` rounded to binary32 and then to the nearest IEEE binary16 value (ties to even, overflow
    to infinity, gradual underflow), as fp64."""
    with np.errstate(over="ignore"):
        return np.asarray(a, dtype=np.float32).astype(np.float16).astype(np.float64).reshape(np.shape(a))
