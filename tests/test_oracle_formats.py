"""Pins for the oracle's scalar formats: E2M1, E4M3, bf16 rounding.

Pinned against (a) hand-computed tables under tests/golden/, (b) torch's float8_e4m3fn and
bfloat16 casts, (c) the CUDA toolkit's host conversion routines (cuda_fp4.h / cuda_fp8.h),
compiled here with nvcc -- three implementations none of which shares code with the oracle.
"""
import ctypes as C
import os
import shutil
import subprocess

import numpy as np
import pytest
import torch

from oracle import pq_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))
GOLD = os.path.join(HERE, "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


def _num(tok):
    if ":" in tok:
        a, b = tok.split(":")
        return float(np.float32(float(a)) * np.float32(2.0) ** int(b))
    return float(np.float32(float(tok)))


def test_e2m1_value_set():
    assert [O.e2m1_value(c) for c in range(8)] == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert [O.e2m1_value(c | 8) for c in range(1, 8)] == [-0.5, -1, -1.5, -2, -3, -4, -6]


def test_e2m1_golden_table():
    for line in _rows("e2m1_roundings.txt"):
        x, code = line.split()
        assert O.e2m1_encode_abs(_num(x)) == int(code), line


def test_e4m3_golden_table():
    for line in _rows("e4m3_roundings.txt"):
        x, code = line.split()
        assert O.e4m3_encode(_num(x)) == int(code, 16), line


def test_e4m3_value_formula():
    # normal: 2^(e-7) (1 + m/8); subnormal: 2^-6 m/8
    for code in range(0x7F):
        e, m = code >> 3, code & 7
        want = 2.0 ** -6 * m / 8 if e == 0 else 2.0 ** (e - 7) * (1 + m / 8)
        assert O.e4m3_value(code) == want
    assert O.e4m3_value(0x7E) == 448.0
    # every representable value encodes to itself
    for code in range(0x7F):
        assert O.e4m3_encode(O.e4m3_value(code)) == code


def test_e4m3_matches_torch_cast():
    """torch's float8_e4m3fn cast is an independent RNE implementation (in range: it does not
    saturate, so only u <= 448 is compared)."""
    rng = np.random.default_rng(0)
    u = np.concatenate([
        rng.uniform(0, 448, 20000), rng.uniform(0, 2.0 ** -5, 20000), rng.uniform(0, 4, 20000),
        np.array([O.e4m3_value(c) for c in range(0x7F)]),
        np.array([(O.e4m3_value(c) + O.e4m3_value(c + 1)) / 2 for c in range(0x7E)]),
    ]).astype(np.float32)
    ref = torch.from_numpy(u).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([O.e4m3_encode(float(v)) for v in u], dtype=np.uint8)
    assert np.array_equal(got, ref)


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-8, 8, 5000),
                        [1.0, 1.00390625, 1.01171875, 0.0, -0.0, 3.0e38]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f32_to_bf16(x), ref)
    assert np.array_equal(O.bf16_to_f32(ref),
                          torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy())


@pytest.fixture(scope="module")
def toolkit_pin(tmp_path_factory):
    if shutil.which("nvcc") is None:
        pytest.skip("nvcc not found: the toolkit's conversion routines cannot be compiled")
    out = str(tmp_path_factory.mktemp("pin") / "libpin.so")
    subprocess.run(["nvcc", "-Wno-deprecated-gpu-targets", "-shared", "-Xcompiler", "-fPIC", "-o", out,
                    os.path.join(HERE, "pin_cuda_fp.cu")], check=True, capture_output=True)
    L = C.CDLL(out)
    for f in (L.pin_e2m1, L.pin_e4m3):
        f.argtypes = [C.c_float]
        f.restype = C.c_ubyte
    return L


def test_e2m1_matches_toolkit_on_every_bf16(toolkit_pin):
    """All finite bf16 bit patterns: sign + magnitude code equals the toolkit's E2M1 cast."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = O.bf16_to_f32(bits)
    for b, v in zip(bits, vals):
        if not np.isfinite(v):
            continue
        mine = (8 if (b & 0x8000) else 0) | O.e2m1_encode_abs(abs(float(v)))
        assert mine == toolkit_pin.pin_e2m1(float(v)), (hex(b), v)


def test_e2m1_matches_toolkit_dense_grid(toolkit_pin):
    """fp32 inputs straddling every rounding boundary by one ulp."""
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32)
    pts = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(9)),
                          np.linspace(0, 8, 4001, dtype=np.float32)])
    for v in pts:
        assert O.e2m1_encode_abs(float(v)) == toolkit_pin.pin_e2m1(float(v)), v


def test_e4m3_matches_toolkit(toolkit_pin):
    rng = np.random.default_rng(2)
    vals = [O.e4m3_value(c) for c in range(0x7F)]
    mids = np.array([(vals[c] + vals[c + 1]) / 2 for c in range(0x7E)], dtype=np.float32)
    pts = np.concatenate([
        np.array(vals, dtype=np.float32), mids, np.nextafter(mids, np.float32(0)),
        np.nextafter(mids, np.float32(1e9)), rng.uniform(0, 600, 30000).astype(np.float32),
        rng.uniform(0, 0.05, 30000).astype(np.float32),
        np.array([448, 464, 465, 480, 1e6, 1e30, 1e-30, 1e-40], dtype=np.float32)])
    for v in pts:
        assert O.e4m3_encode(float(v)) == toolkit_pin.pin_e4m3(float(v)), v
