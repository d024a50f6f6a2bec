"""Pins for the oracle's output-side calibration error (Sec. 3.3, the error behind the acceptance
rule of Eq. 10 read on the layer's output): closed forms, a float64 sum, the stated summation
order written out with numpy scalars, and its tie to the input-side group error of Eq. 3."""
import numpy as np
import torch

from oracle import pq_oracle as O
from paper_2605_09503_b200 import inputs


def bf(a):
    return inputs.bits(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def test_equal_outputs_have_zero_error_and_nothing_is_accumulated():
    y = np.arange(300 * 8, dtype=np.float32).reshape(300, 8) % 97 - 48.0      # exact in bf16
    err = O.output_error(y, bf(y), np.full(8, 3.25))
    assert np.array_equal(err, np.full(8, 3.25))


def test_constant_difference_closed_form():
    rows, N = 333, 16
    c = np.array([0.5, -1, 2, 3, -4, 0, 1.5, 8, 0.25, -0.75, 16, 1, -2, 5, 6, -7], dtype=np.float32)
    yq = (np.arange(rows)[:, None] % 5 - 2.0) * np.ones(N, dtype=np.float32)
    err = O.output_error(yq + c[None, :], bf(yq))
    assert np.array_equal(err, rows * c.astype(np.float64) ** 2)     # exact: small dyadic numbers


def test_against_float64_sum_and_accumulation_over_batches():
    g = np.random.default_rng(5)
    rows, N = 150, 40
    total = np.zeros(N)
    err = None
    for _ in range(2):
        yref = g.standard_normal((rows, N)).astype(np.float32) * 7
        yq = bf(yref + 0.3 * g.standard_normal((rows, N)).astype(np.float32))
        err = O.output_error(yref, yq, err)
        d = (yref - O.bf16_to_f32(yq)).astype(np.float64)            # the fp32 difference, then fp64
        total += (d ** 2).sum(axis=0)
    assert np.allclose(err, total, rtol=1e-6, atol=0)
    assert not np.allclose(err, total / 2, rtol=0.2)


def test_transposed_or_swapped_operands_are_told_apart():
    """Column n of err belongs to column n of the outputs, and the bf16 operand is the second one."""
    rows, N = 20, 8
    yref = np.zeros((rows, N), dtype=np.float32)
    yq = np.zeros((rows, N), dtype=np.float32)
    yq[:, 3] = 2.0
    yq[7, 5] = 1.0
    err = O.output_error(yref, bf(yq))
    want = np.zeros(N)
    want[3], want[5] = 4.0 * rows, 1.0
    assert np.array_equal(err, want)
    # a value that bf16 cannot hold distinguishes the fp32 operand from the bf16 one
    fine = np.full((4, 8), 1.0 + 2.0 ** -12, dtype=np.float32)
    assert np.array_equal(O.output_error(fine, bf(np.ones((4, 8)))), np.full(8, 4 * 2.0 ** -24))


def _fold(d, rows, chunk=16, slab=128):
    """Column sums of squares of float32 d in the stated order, written out with numpy scalars."""
    want = np.zeros(d.shape[1])
    for s0 in range(0, rows, slab):
        acc = np.zeros(d.shape[1])
        for r0 in range(s0, min(s0 + slab, rows), chunk):
            p = np.zeros(d.shape[1], dtype=np.float32)
            for t in range(r0, min(r0 + chunk, s0 + slab, rows)):
                p = (p.astype(np.float64) + d[t].astype(np.float64) ** 2).astype(np.float32)   # = fmaf
            acc += p.astype(np.float64)
        want += acc
    return want


def test_summation_order_is_the_stated_one():
    """Chunks of 16 rows in fp32 (fused multiply-add), slabs of 128 rows in fp64 from zero, slab sums
    in order; the difference itself is one fp32 subtraction."""
    g = np.random.default_rng(11)
    rows, N = 300, 24
    yref = (g.standard_normal((rows, N)) * np.exp(g.standard_normal((rows, N)) * 3)).astype(np.float32)
    yq = bf(yref * (1 + 0.1 * g.standard_normal((rows, N)).astype(np.float32)))
    d = yref - O.bf16_to_f32(yq)                                      # float32 - float32 -> float32
    want = _fold(d, rows)
    got = O.output_error(yref, yq)
    assert np.array_equal(got, want)
    # the order matters on this input: a flat float64 sum gives other bits somewhere
    assert not np.array_equal(got, (d.astype(np.float64) ** 2).sum(axis=0))


def test_identity_layer_output_error_is_the_input_group_error():
    """With W = I (exactly representable in NVFP4) the quantized layer's output is the dequantized
    activation, so the output-side error summed over columns is the input-side error of Eq. 3
    summed over groups: two routes through different oracle functions."""
    cfg = inputs.CONFIGS["tiny"]
    K = 64
    x = np.ascontiguousarray(inputs.bits(inputs.activations(cfg, 0, 0, rows=96))[:, :K])
    ts = float(np.abs(O.bf16_to_f32(x)).max()) / 2688.0
    codes, sf = O.quant_nvfp4(x, ts)
    xhat = O.dequant_nvfp4(codes, sf, ts)                             # float64 [rows, K], exact values
    # dequantized values are products of three short floats: exactly representable in float32
    assert np.array_equal(xhat, xhat.astype(np.float32).astype(np.float64))
    # the bf16 operand of output_error is Yq, so hand it the exact activations and let Yref carry
    # the dequantized ones: the squares are the same
    e_out = O.output_error(xhat.astype(np.float32), x).sum()
    e_in = O.group_error(x, 0, 4, 16, ts=ts).sum()
    assert np.isclose(e_out, e_in, rtol=1e-5, atol=0)
