"""The layer table and input generators against the values the paper prints (CPU only)."""
import os

import numpy as np

from paper_2609_10632_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_structural_pins.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def test_layer_table_matches_paper_counts():
    gold = _golden()
    layers = wl.detector_layers(int(gold["batch"]), 640)
    assert len(layers) == 77
    conv_bn = sum(s.kdim * s.c_out + 2 * s.c_out for s in layers)
    plain = sum(ci * co + co for ci, co in wl.detector_plain_head_convs())
    total = conv_bn + plain
    assert conv_bn == 25_843_824 and plain == 58_800
    assert round(total / 1e6, 1) == gold["params_millions"]
    # trainable tensors: weight + gamma + beta per Conv-BN-SiLU layer, weight + bias per plain head conv
    assert 3 * len(layers) + 2 * len(wl.detector_plain_head_convs()) == int(gold["gradient_tensors"])
    tensors = wl.detector_parameter_tensors()  # the optimiser's tensor list
    assert len(tensors) == int(gold["gradient_tensors"]) and sum(n for _, n, _ in tensors) == total
    assert [sum(1 for t in tensors if t[2] == g) for g in (0, 1, 2)] == [83, 77, 83]  # decayed weights, BN gains, biases
    # head levels
    heads = [s for s in layers if s.name.startswith("h22.cls") and s.name.endswith(".0")]
    assert sum(s.ho * s.wo for s in heads) == int(gold["candidate_locations"])
    assert sorted(640 // s.h for s in heads) == [8, 16, 32]
    box = [s for s in layers if s.name.startswith("h22.box")]
    assert all(s.c_out == 4 * int(gold["reg_max"]) for s in box)
    assert [co for _, co in wl.detector_plain_head_convs()][1] == int(gold["classes"])
    assert len(wl.distinct_shapes(layers)) == 35
    assert sum(m for _, m in wl.distinct_shapes(layers)) == 77
    flops = sum(s.gemm_flops for s in layers)
    assert abs(flops / 16 / 1e9 - 78.61) < 0.01


def test_config_shapes():
    c1, = wl.config_shapes(1)
    assert (c1.m, c1.kdim, c1.c_out) == (2048, 144, 32)
    c2, = wl.config_shapes(2)
    assert (c2.m, c2.kdim, c2.ho) == (1_638_400, 27, 320) and c2.image_input
    c3, = wl.config_shapes(3)
    assert (c3.m, c3.kdim) == (409_600, 864)
    a, b = wl.config_shapes(4)
    assert (a.m, a.kdim, b.m, b.kdim, b.ho) == (25_600, 384, 25_600, 1728, 40)
    assert len(wl.config_shapes(5)) == 77


def test_bf16_rounding_is_rne_and_idempotent():
    vals = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7 + 2 ** -8, 1.0 + 2 ** -8 + 2 ** -20, -3.1415926, 0.0, 65280.0], dtype=np.float32)
    r = wl.round_to_bf16(vals)
    assert r[0] == 1.0
    assert r[1] == 1.0  # tie -> even mantissa
    assert r[2] == np.float32(1.0 + 2 ** -6)  # tie -> even (up)
    assert r[3] == np.float32(1.0 + 2 ** -7)  # above the tie -> up
    assert abs(r[4] + 3.140625) < 1e-6
    np.testing.assert_array_equal(wl.round_to_bf16(r), r)
    bits = wl.f32_to_bf16_bits(vals)
    assert bits.dtype == np.uint16
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(bits), r)


def test_generators_seeded_and_distributed_as_stated():
    gold = _golden()
    s = wl.ConvShape("t", 2, 32, 32, 16, 32, 3, 1)
    a = wl.make_inputs(s, 1, 0, bf16=False)
    b = wl.make_inputs(s, 1, 0, bf16=False)
    np.testing.assert_array_equal(a.x, b.x)
    np.testing.assert_array_equal(a.w, b.w)
    c = wl.make_inputs(s, 1, 1, bf16=False)
    assert not np.array_equal(a.x, c.x)
    bound = 1 / np.sqrt(16 * 9)
    assert np.abs(a.w).max() <= bound and np.abs(a.w).max() > 0.95 * bound
    # Kaiming-uniform(a=sqrt 5): std = bound/sqrt 3; Kaiming-normal(gain sqrt 2): std = sqrt(2/fan_in); ratio sqrt 6
    big = wl.make_inputs(wl.ConvShape("t", 1, 8, 8, 64, 256, 3, 1), 1, 2, bf16=False)
    std_u = big.w.std()
    std_n = np.sqrt(2.0 / (64 * 9))
    assert abs(std_n / std_u - gold["kaiming_normal_over_uniform"]) < 0.02
    assert abs(a.x.mean()) < 0.02 and abs(a.x.std() - 1) < 0.02
    img = wl.make_inputs(wl.ConvShape("t", 1, 64, 64, 3, 48, 3, 2, True), 2, 0)
    assert img.x.min() >= 0 and img.x.max() <= 1 and abs(img.x.mean() - 0.5) < 0.02
    np.testing.assert_array_equal(wl.round_to_bf16(img.x), img.x)
    assert np.all(a.gamma == 1) and np.all(a.beta == 0)
    r = wl.make_inputs(s, 1, 0, affine="random")
    assert r.gamma.min() >= 0.5 and r.gamma.max() <= 1.5 and np.abs(r.beta).max() < 1
