"""The kernels evaluate the quantiser without the IEEE division sequence (reciprocal +
two fused multiply-adds, with the division as fallback near rounding ties).  This checks,
on the device and over every finite FP32 input, that the shortcut returns the same code
as clamp(round_half_even(x / s)) for a spread of scales and bit widths."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _scales():
    rng = np.random.default_rng(7)
    s = [1.0, 0.5, 2.0 ** -10, 3.0, 1.0 / 3.0, 0.1, 1e-8 / 7, 1e-8 / 127, 7.25e-4, 4.4e-3,
         np.float32(1) - np.float32(2.0 ** -24),            # mantissa all ones
         np.float32(2) - np.float32(2.0 ** -23), 1e-30, 1e30, 1e-36, 1e36, 2.0 ** -100, 2.0 ** 100]
    s += list(np.exp(rng.uniform(np.log(1e-6), np.log(10.0), 22)))
    return [float(np.float32(x)) for x in s]


def test_division_free_quantiser_equals_definition_for_all_inputs():
    import torch
    import paper_2410_20046_b200 as dq

    ctx = dq.Context([0, 4], 16, 16, 16)
    bad = torch.zeros(1, dtype=torch.int64, device="cuda")
    scales = _scales()
    for k, s in enumerate(scales):
        bits = (2, 4, 8, 16)[k % 4]
        ctx.selfcheck_quantizer(s, bits, 0, 1 << 32, bad)          # all 2^32 bit patterns
        assert int(bad.item()) == 0, f"scale {s!r} bits {bits}: {int(bad.item())} codes differ"
    for bits in (3, 4, 8):                                          # every width on the training scales
        for s in scales[6:10]:
            ctx.selfcheck_quantizer(s, bits, 0, 1 << 32, bad)
    assert int(bad.item()) == 0
    ctx.close()
