"""The seeded input generators: Philox known answers, bf16 rounding, neighbour tables."""
import os

import numpy as np
import torch

from vvs_synth import gen, philox
from vvs_synth.configs import CONFIGS, XL

HERE = os.path.dirname(os.path.abspath(__file__))


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        got = philox.philox4x32_10(np.array([w[0:4]], np.uint32), np.array([w[4:6]], np.uint32))[0]
        assert [int(x) for x in got] == w[6:10]


def test_uniforms_are_open_interval_and_reproducible():
    u = philox.verify_uniforms(0x56565301, 7, 16, 8)
    assert u.shape == (16, 9) and u.dtype == np.float32
    assert (u > 0).all() and (u < 1).all()
    np.testing.assert_array_equal(u, philox.verify_uniforms(0x56565301, 7, 16, 8))
    assert (u != philox.verify_uniforms(0x56565301, 8, 16, 8)).any()
    big = philox.verify_uniforms(1, 0, 512, 63)
    assert abs(big.mean() - 0.5) < 0.01
    assert philox.uniform_open01(np.array([0, 0xFFFFFFFF], np.uint32)).tolist() == \
        [np.float32(2.0 ** -25), np.float32(1 - 2.0 ** -25)]


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 3
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gen.f32_to_bf16_bits(x), want)
    np.testing.assert_array_equal(gen.bf16_bits_to_f32(want),
                                  torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_neighbour_table_is_exact_topk_self_first():
    e = gen.make_codebook(3, 300, 8)
    e[17] = e[5]                                               # duplicate code: distance tie
    row_ptr, col = gen.neighbour_csr(e, 9)
    col = col.reshape(300, 9)
    np.testing.assert_array_equal(row_ptr, np.arange(301) * 9)
    for x in (0, 5, 17, 123, 299):
        d = ((e - e[x]) ** 2).sum(1)
        d[x] = -1
        order = sorted(range(300), key=lambda y: (d[y], y))
        assert list(col[x]) == order[:9]
        assert col[x, 0] == x
    assert col[17, 1] == 5 and col[5, 1] == 17


def test_streamed_parameter_counts():
    """Per-step weight traffic used by the roofline: 36 x 19.82 M + 20.97 M parameters."""
    assert XL.params_per_layer == 19_824_640
    assert XL.streamed_params == 36 * 19_824_640 + 16384 * 1280
    assert CONFIGS[2].n_rows == 32 and CONFIGS[1].block_len == 9
