"""The cubic that replaces a share of the exp2 instructions in the dQ kernel (csrc/sm100.cuh,
ex2_fma_pair): its coefficients are read from the source and checked against 2^f on [0, 1) in the
arithmetic the kernel uses (fp32 Horner steps with fused multiply-adds), together with the
reconstruction 2^x = 2^floor(x) * 2^(x - floor(x)) over the range of arguments the kernel clamps to."""
import os
import re

import numpy as np

SRC = os.path.join(os.path.dirname(__file__), "..", "paper_2608_25683_b200", "csrc", "sm100.cuh")


def coefficients():
    text = open(SRC).read()
    body = text[text.index("ex2_fma_pair"):]
    c = [float(re.search(r"c%d = make_f32x2\(([0-9.eE+-]+)f" % i, body).group(1)) for i in (1, 2, 3)]
    clamp = float(re.search(r"fmaxf\(x0, (-[0-9.]+)f\)", body).group(1))
    magic = float(re.search(r"magic = make_f32x2\(([0-9.]+)f", body).group(1))
    return c, clamp, magic


def cubic(f, c):
    f = np.asarray(f).astype(np.float32).astype(np.float64)
    c1, c2, c3 = (np.float32(x) for x in c)
    # fp64 products rounded once to fp32 = fused multiply-add
    p = (np.float64(c3) * f + np.float64(c2)).astype(np.float32)
    p = (p.astype(np.float64) * f + np.float64(c1)).astype(np.float32)
    p = (p.astype(np.float64) * f + 1.0).astype(np.float32)
    return p


def test_cubic_error_on_unit_interval():
    c, _, _ = coefficients()
    f = np.linspace(0.0, 1.0, 200001, dtype=np.float64)[:-1]
    rel = np.abs(cubic(f, c).astype(np.float64) / np.exp2(f.astype(np.float32).astype(np.float64)) - 1.0)
    assert rel.max() < 1e-4, rel.max()          # 8.6e-5 by construction; bf16 keeps 2^-9 = 2e-3
    assert cubic(np.array([0.0]), c)[0] == np.float32(1.0)


def test_reconstruction_over_the_clamped_range():
    c, clamp, magic = coefficients()
    assert clamp == -126.0 and magic == 12582912.0      # 1.5 * 2^23: floor(x) sits in the low mantissa bits
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.uniform(-126.0, 1.0, 100000), [-126.0, -1.0, 0.0, -0.5, 0.999]]).astype(np.float32)
    n = np.floor(x)
    t_bits = (np.float32(magic).view(np.int32).astype(np.int64) + n.astype(np.int64))   # bits of x + magic, rounded down
    p_bits = cubic((x - n).astype(np.float64), c).view(np.int32).astype(np.int64)
    r_bits = (p_bits + ((t_bits << 23) & 0xFFFFFFFF)) & 0xFFFFFFFF
    r = r_bits.astype(np.uint32).view(np.float32).astype(np.float64)
    ref = np.exp2(x.astype(np.float64))
    assert np.all(np.isfinite(r))
    assert np.abs(r / ref - 1.0).max() < 1.2e-4
