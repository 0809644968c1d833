"""Pins for the bfloat16 scale / bias variant of the format (Section 3.2 and Appendix "safetensors Q4 Format" name
bfloat16 for two of the three models and float16 for the third).  CPU only.

The oracle's directed roundings are checked against a search over the table of all finite bfloat16 values, the
quantizer against hand-worked literals and exact rational arithmetic, the container against an independent reader."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth


def bf16(x):
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


def _all_finite_bf16():
    bits = np.arange(65536, dtype=np.uint32)
    vals = (bits << np.uint32(16)).view(np.float32)
    keep = np.isfinite(vals)
    bits, vals = bits[keep], vals[keep].astype(np.float64)
    order = np.argsort(vals, kind="stable")
    return bits[order].astype(np.uint16), vals[order]


def test_directed_roundings_against_a_search_over_all_bf16_values():
    bits, vals = _all_finite_bf16()
    g = synth.rng(31, 0)
    x = np.concatenate([
        g.standard_normal(4000).astype(np.float32) * np.float32(3.0),
        (g.standard_normal(2000) * 1e-3).astype(np.float32),
        (g.standard_normal(2000) * 2e4).astype(np.float32),
        np.array([0.2, -0.2, 1.0, -1.0, 65504.0, -65504.0, 1e-30, -1e-30, 0.19921875, 0.2001953125], dtype=np.float32),
    ])
    x = x[np.abs(x) <= 65504.0]
    down = O._bf16_round_down(x)
    up = O._bf16_round_up(x)
    x64 = x.astype(np.float64)
    # largest table value <= x, smallest table value >= x (+0 and -0 are equal as numbers: compare values)
    i_dn = np.searchsorted(vals, x64, side="right") - 1
    i_up = np.searchsorted(vals, x64, side="left")
    assert np.array_equal(O.sb_values(down), vals[i_dn])
    assert np.array_equal(O.sb_values(up), vals[i_up])
    assert np.all(O.sb_values(down) <= x64) and np.all(O.sb_values(up) >= x64)
    exact = (x.view(np.uint32) & 0xFFFF) == 0
    assert np.array_equal(down[exact], (x.view(np.uint32) >> 16).astype(np.uint16)[exact])
    assert np.array_equal(up[exact], down[exact])


def test_sb_values_reads_both_types():
    assert O.sb_values(np.array([0x3F80, 0xBF80, 0x3E4D, 0x0000], dtype=np.uint16)).tolist() == [1.0, -1.0, 0.2001953125, 0.0]
    assert O.sb_values(np.array([1.5, -0.25], dtype=np.float16)).tolist() == [1.5, -0.25]


def test_literal_scale_rounds_up_bias_is_the_minimum():
    # min -1, max 2: r = 3, r / 15 = 0.2 = 0x3E4CCCCD in binary32; its bfloat16 neighbours are 0x3E4C (0.19921875) and
    # 0x3E4D (0.2001953125): nearest would also give 0x3E4D here, so a second group pins the direction:
    # min 0, max 1.5: r / 15 = 0.1 = 0x3DCCCCCD, neighbours 0x3DCC (0.099609375) and 0x3DCD (0.10009765625): nearest is
    # 0x3DCD as well; min 0, max 0.75: 0.05 = 0x3D4CCCCD -> 0x3D4D.  A value just above a table entry separates them:
    # min 0, max 15 * 0.125 + 2^-7: r / 15 = 0.12552..., nearest is 0x3E00 (0.125), round-up 0x3E01 (0.1259765625).
    g = np.full((2, 64), -1.0, dtype=np.float32)
    g[0, :5] = [2.0, 0.5, 0.0, 1.25, -1.0]
    g[1] = 0.0
    g[1, 0] = 15 * 0.125 + 2.0**-7
    g[1, 1] = 0.125 * 7.4
    g = bf16(g)
    c, s, b = O.quantize_rows(g, sb_dtype=1)
    assert s.dtype == np.uint16 and b.dtype == np.uint16
    assert s[0, 0] == 0x3E4D and b[0, 0] == 0xBF80
    # t = (x + 1) / 0.2001953125: 14.985 -> 15, 7.49 -> 7, 4.995 -> 5, 11.24 -> 11, 0 -> 0
    assert list(c[0, :5]) == [15, 7, 5, 11, 0]
    assert s[1, 0] == 0x3E01 and b[1, 0] == 0x0000
    assert c[1, 0] == 15                                    # 1.8828125 / 0.1259765625 = 14.95


def test_bias_equals_the_group_minimum_and_minus_zero_becomes_plus_zero():
    x = bf16(synth.rng(32, 0).standard_normal((8, 128), dtype=np.float32) * 5)
    c, s, b = O.quantize_rows(x, sb_dtype=1)
    mn = x.reshape(8, 2, 64).min(axis=-1)
    assert np.array_equal(b, synth.f32_to_bf16_bits(mn))   # the inputs are bfloat16 already: nothing to round
    g = np.zeros((1, 64), dtype=np.float32)
    g[0, 0] = -0.0
    g[0, 1] = 3.0
    c, s, b = O.quantize_rows(g, sb_dtype=1)
    assert b[0, 0] == 0x0000


def test_ties_go_to_even_and_unit_scale():
    g = np.zeros(64, dtype=np.float32)
    g[:8] = [0.0, 15.0, 0.5, 1.5, 2.5, 3.5, 7.0, 14.5]
    c, s, b = O.quantize_rows(g[None, :], sb_dtype=1)
    assert s[0, 0] == 0x3F80 and b[0, 0] == 0
    assert list(c[0, :8]) == [0, 15, 0, 2, 2, 4, 7, 14]


def test_half_step_bound_in_exact_arithmetic():
    g = synth.rng(33, 0)
    x = g.standard_normal((6, 128), dtype=np.float32)
    x[1] *= 100.0
    x[2] = 1000.0 + 0.01 * x[2]
    x[3, :64] = 3.0
    x[4] *= 1e-6
    x[5, 5] = 65280.0
    x[5, 6] = -65280.0
    x = bf16(x)
    c, s, b = O.quantize_rows(x, sb_dtype=1)
    sv, bv = O.sb_values(s), O.sb_values(b)
    for row in range(6):
        for gi in range(2):
            sc, bi = Fraction(float(sv[row, gi])), Fraction(float(bv[row, gi]))
            for i in range(64):
                xv = Fraction(float(x[row, gi * 64 + i]))
                xh = int(c[row, gi * 64 + i]) * sc + bi
                assert abs(xv - xh) <= sc / 2 * (1 + Fraction(1, 100000)), (row, gi, i)
    # the scale's range covers the group: bias + 15 scale >= max
    mx = x.reshape(6, 2, 64).max(axis=-1).astype(np.float64)
    assert np.all(bv + 15 * sv >= mx)
    xh = O.dequantize(c, s, b)
    assert xh[0, 3] == float(int(c[0, 3]) * Fraction(float(sv[0, 0])) + Fraction(float(bv[0, 0])))


def test_affine_ladder_encodes_to_its_own_indices():
    for bias, step in [(0.0, 1.0), (-4.0, 0.5), (0.25, 0.0625), (-30.0, 4.0)]:
        ladder = bias + step * np.arange(16, dtype=np.float32)
        x = np.tile(ladder, 4)[None, :]
        assert np.array_equal(bf16(x), x)
        c, s, b = O.quantize_rows(x, sb_dtype=1)
        assert O.sb_values(s)[0, 0] == step and O.sb_values(b)[0, 0] == bias
        assert np.array_equal(c[0], np.tile(np.arange(16), 4))
        assert np.array_equal(O.dequantize(c, s, b), x.astype(np.float64))


def test_both_types_agree_where_both_roundings_are_exact():
    # scale and bias representable in binary16 and bfloat16 alike: same codes, same values
    x = np.tile(-2.0 + 0.25 * np.arange(16, dtype=np.float32), 4)[None, :]
    c0, s0, b0 = O.quantize_rows(x, sb_dtype=0)
    c1, s1, b1 = O.quantize_rows(x, sb_dtype=1)
    assert np.array_equal(c0, c1)
    assert np.array_equal(O.sb_values(s0), O.sb_values(s1)) and np.array_equal(O.sb_values(b0), O.sb_values(b1))


def test_pool_append_gather_and_byte_counts():
    spec = O.Spec(1, 4, 2, 128, 128, sb_dtype=1)
    assert spec.packed_bytes(300) == O.Spec(1, 4, 2, 128, 128).packed_bytes(300)
    pool = O.Pool(spec, 3)
    assert pool.Ks.dtype == np.uint16 and pool.Vb.dtype == np.uint16
    g = synth.rng(34, 0)
    k = bf16(g.standard_normal((5, 2, 128), dtype=np.float32))
    v = bf16(g.standard_normal((5, 2, 128), dtype=np.float32))
    O.quantize_append(pool, 0, [[2, 0]], [254], [0, 5], k, v)          # crosses a block edge
    K, V = O.gather_dequant(pool, 0, [2, 0], 254, 259, 1)
    c, s, b = O.quantize_rows(k[:, 1], sb_dtype=1)
    assert np.array_equal(K, O.dequantize(c, s, b))
    assert np.max(np.abs(K - k[:, 1])) <= 0.5 * O.sb_values(s).max() * (1 + 1e-6)
    buf = O.pack(pool, [2, 0], 259)
    pool2 = O.Pool(spec, 3)
    O.unpack(pool2, [1, 2], 259, buf)
    K2, V2 = O.gather_dequant(pool2, 0, [1, 2], 254, 259, 1)
    assert np.array_equal(K, K2) and np.array_equal(V, V2)


def test_container_names_the_type_and_opens_with_an_independent_reader():
    st = pytest.importorskip("safetensors.torch")
    import torch
    spec = O.Spec(2, 4, 2, 128, 128, sb_dtype=1)
    pool = O.Pool(spec, 3)
    g = synth.rng(35, 0)
    for t in pool.tensors():
        if t.dtype == np.uint32:
            t[:] = g.integers(0, 2**32, size=t.shape, dtype=np.uint64).astype(np.uint32)
        else:
            t[:] = synth.f32_to_bf16_bits(g.standard_normal(t.shape).astype(np.float32))
    image = O.container(pool, [2, 0], 300).tobytes()
    tensors = st.load(image)
    assert len(tensors) == 2 * 2 * 6
    t = tensors["L1_B1_V_scales"]
    assert t.dtype == torch.bfloat16 and tuple(t.shape) == (2, 256, 2)
    want = pool.Vs[1, 0].copy()
    want[:, 300 - 256:] = 0
    assert np.array_equal(t.view(torch.int16).numpy().view(np.uint16), want)
    assert np.array_equal(t.float().numpy().astype(np.float64), O.sb_values(want))
    n = int.from_bytes(image[:8], "little")
    assert b'"sb_dtype":"1"' in image[8:8 + n] and b'"dtype":"BF16"' in image[8:8 + n]
