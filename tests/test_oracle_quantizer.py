"""Pins for the oracle's quantizer and packed layout (CPU only).

Each test fixes the oracle to something other than itself: closed forms,
hand-worked literals, exact arithmetic in Fractions, the paper's byte counts.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_kv_bytes.txt")


def bf16(x):
    """float -> nearest bf16 -> float32 (test inputs must be bf16-representable)."""
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


# ---- layout / byte counts against the paper's printed numbers -------------------------------
def _golden_rows():
    rows, ratio = [], None
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[0] == "ratio":
            ratio = float(f[1])
        else:
            rows.append(f)
    return rows, ratio


def test_packed_bytes_match_paper_tables():
    rows, ratio = _golden_rows()
    assert ratio == 0.28125
    for name, L, H, dk, dv, n, code_b, sb_b, layer_b, mib in rows:
        L, H, dk, dv, n = int(L), int(H), int(dk), int(dv), int(n)
        spec = O.Spec(L, H, H, dk, dv)
        total = spec.packed_bytes(n)
        assert total == float(mib) * 2**20, name
        fp16 = L * H * (dk + dv) * n * 2
        assert total / fp16 == ratio
        if layer_b != "-":
            assert total // L == int(layer_b)
            assert H * n * (dk + dv) // 2 == int(code_b)          # packed nibbles
            assert H * n * 4 * (dk + dv) // 64 == int(sb_b)       # fp16 scale + bias per group


def test_pack_buffer_has_paper_size_and_zero_tail():
    spec = O.Spec(2, 4, 2, 128, 128)
    pool = O.Pool(spec, 5, fill=0xFFFFFFFF)
    pool.Ks[:] = 1.0
    buf = O.pack(pool, [3, 1], 300)
    assert buf.size == 2 * 2 * 256 * 2 * (64 + 8 + 64 + 8)
    # formula h*d*n*(1+8/g) per layer for K+V, n = whole blocks
    assert buf.size == 2 * int(2 * 128 * 512 * (1 + 8 / 64))
    # slots >= 300 (block 1, slot 44 on) are zero bytes in every tensor
    blk = buf[spec.block_bytes():2 * spec.block_bytes()]
    kc = blk[:2 * 256 * 64].view(np.uint32).reshape(2, 256, 16)
    assert np.all(kc[:, 44:] == 0) and np.all(kc[:, :44] == 0xFFFFFFFF)


def test_pack_tensor_order_and_byte_offsets_are_literal():
    """Appendix A order inside one persisted block: K codes, K scales, K biases, V codes, V scales, V biases, each
    [Hkv][256][...] row-major.  Every tensor carries its own sentinel, and the offsets below are typed out for
    Hkv 2, d_qk 128, d_v 64: K codes 2*256*64 = 32768 B, K scales / biases 2*256*2*2 = 2048 B each, V codes
    2*256*32 = 16384 B, V scales / biases 2*256*1*2 = 1024 B each; block = 55296 B; two layers, two blocks each."""
    spec = O.Spec(2, 2, 2, 128, 64)
    pool = O.Pool(spec, 3)
    pool.Kc[:] = 0x11111111
    pool.Ks[:] = np.float16(2.0)       # 0x4000
    pool.Kb[:] = np.float16(-3.0)      # 0xC200
    pool.Vc[:] = 0x44444444
    pool.Vs[:] = np.float16(5.0)       # 0x4500
    pool.Vb[:] = np.float16(-6.0)      # 0xC600
    # single elements that name their own coordinates: (layer 1, physical block 0 = logical block 1, head 1, slot 7)
    pool.Kc[1, 0, 1, 7, 3] = 0xA1B2C3D4
    pool.Ks[1, 0, 1, 7, 1] = np.float16(0.5)    # 0x3800
    pool.Kb[1, 0, 1, 7, 0] = np.float16(0.25)   # 0x3400
    pool.Vc[1, 0, 1, 7, 2] = 0x0BADF00D
    pool.Vs[1, 0, 1, 7, 0] = np.float16(0.125)  # 0x3000
    pool.Vb[1, 0, 1, 7, 0] = np.float16(64.0)   # 0x5400
    buf = O.pack(pool, [2, 0], 512)
    assert spec.block_bytes() == 55296 and buf.size == 4 * 55296
    u16 = lambda off: int(buf[off]) | int(buf[off + 1]) << 8
    u32 = lambda off: u16(off) | u16(off + 2) << 16
    for blk in range(4):                                        # tensor starts inside every block
        base = blk * 55296
        assert u32(base) == 0x11111111 and u32(base + 32764) == 0x11111111
        assert u16(base + 32768) == 0x4000 and u16(base + 34814) == 0x4000
        assert u16(base + 34816) == 0xC200 and u16(base + 36862) == 0xC200
        assert u32(base + 36864) == 0x44444444 and u32(base + 53244) == 0x44444444
        assert u16(base + 53248) == 0x4500 and u16(base + 54270) == 0x4500
        assert u16(base + 54272) == 0xC600 and u16(base + 55294) == 0xC600
    base = 3 * 55296                                            # layer 1, logical block 1
    assert u32(base + ((1 * 256 + 7) * 16 + 3) * 4) == 0xA1B2C3D4
    assert u16(base + 32768 + ((1 * 256 + 7) * 2 + 1) * 2) == 0x3800
    assert u16(base + 34816 + ((1 * 256 + 7) * 2 + 0) * 2) == 0x3400
    assert u32(base + 36864 + ((1 * 256 + 7) * 8 + 2) * 4) == 0x0BADF00D
    assert u16(base + 53248 + (1 * 256 + 7) * 2) == 0x3000
    assert u16(base + 54272 + (1 * 256 + 7) * 2) == 0x5400
    # and unpack puts every byte back where it came from
    pool2 = O.Pool(spec, 3)
    O.unpack(pool2, [1, 2], 512, buf)
    assert pool2.Kc[1, 2, 1, 7, 3] == 0xA1B2C3D4 and pool2.Vb[1, 2, 1, 7, 0] == np.float16(64.0)
    assert pool2.Ks[1, 2, 1, 7, 1] == np.float16(0.5) and pool2.Kb[0, 1, 0, 0, 0] == np.float16(-3.0)


# ---- hand-worked literals -------------------------------------------------------------------
def test_literal_unit_scale_and_ties_to_even():
    g = np.zeros(64, dtype=np.float32)
    g[:8] = [0.0, 15.0, 0.5, 1.5, 2.5, 3.5, 7.0, 14.5]
    c, s, b = O.quantize_rows(bf16(g)[None, :])
    assert s[0, 0] == np.float16(1.0) and b[0, 0] == np.float16(0.0)
    assert list(c[0, :8]) == [0, 15, 0, 2, 2, 4, 7, 14]
    assert np.all(c[0, 8:] == 0)


def test_literal_scale_rounds_up_bias_exact():
    # min -1, max 2: r = 3, r/15 = 0.2 -> binary16 neighbours 0x3266 (0.19995117) and 0x3267 (0.20007324);
    # nearest would pick 0x3266, round-up must pick 0x3267.
    g = np.full(64, -1.0, dtype=np.float32)
    g[:5] = [2.0, 0.5, 0.0, 1.25, -1.0]
    c, s, b = O.quantize_rows(g[None, :])
    assert s.view(np.uint16)[0, 0] == 0x3267
    assert b.view(np.uint16)[0, 0] == 0xBC00
    # t = (x+1)/0.20007324: 14.99 -> 15, 7.497 -> 7, 4.998 -> 5, 11.246 -> 11, 0 -> 0
    assert list(c[0, :5]) == [15, 7, 5, 11, 0]


def test_literal_bias_rounds_down_in_subnormal_range():
    tiny = bf16(-2e-8)                   # above -2^-25: nearest binary16 is -0, round-down is -2^-24
    g = np.zeros(64, dtype=np.float32)
    g[0] = tiny.item()
    g[1] = 1.0
    c, s, b = O.quantize_rows(g[None, :])
    assert b.view(np.uint16)[0, 0] == 0x8001
    assert float(b[0, 0]) <= tiny.item()
    assert c[0, 0] == 0 and c[0, 1] == 15


def test_negative_zero_bias_is_stored_as_plus_zero():
    g = np.zeros(64, dtype=np.float32)
    g[0] = -0.0
    g[1] = 3.0
    c, s, b = O.quantize_rows(g[None, :])
    assert b.view(np.uint16)[0, 0] == 0x0000


def test_nibble_order_lsb_first():
    codes = np.arange(16, dtype=np.uint8)[None, :]
    w = O.pack_codes(codes)
    assert w.tolist() == [[0x76543210, 0xFEDCBA98]]
    assert np.array_equal(O.unpack_codes(w), codes)


# ---- invariants in exact arithmetic ---------------------------------------------------------
def _check_half_step(x32, c, s, b):
    D = x32.shape[-1]
    for row in range(x32.shape[0]):
        for gi in range(D // 64):
            sc, bi = Fraction(float(s[row, gi])), Fraction(float(b[row, gi]))
            for i in range(64):
                x = Fraction(float(x32[row, gi * 64 + i]))
                xh = int(c[row, gi * 64 + i]) * sc + bi
                assert abs(x - xh) <= sc / 2 * (1 + Fraction(1, 100000)), (row, gi, i)


def test_half_step_bound_random_and_adversarial():
    g = synth.rng(7, 0)
    x = g.standard_normal((6, 128), dtype=np.float32)
    x[1] *= 100.0
    x[2] = 1000.0 + 0.01 * x[2]              # near-constant group with a large offset
    x[3, :64] = 3.0                           # constant group
    x[4] *= 1e-6                              # tiny magnitudes (binary16 subnormal scale)
    x[5, 5] = 65280.0                          # largest bf16 below the binary16 maximum
    x[5, 6] = -65280.0
    x = bf16(x)
    c, s, b = O.quantize_rows(x)
    assert c.max() <= 15
    _check_half_step(x, c, s, b)
    # dequantize() agrees with the exact rational value
    xh = O.dequantize(c, s, b)
    assert xh[0, 3] == float(int(c[0, 3]) * Fraction(float(s[0, 0])) + Fraction(float(b[0, 0])))


@pytest.mark.parametrize("v", [0.0, 1.0, -2.5, 0.15625, 30.0])
def test_all_equal_group_encodes_exactly(v):
    x = np.full((1, 64), v, dtype=np.float32)
    c, s, b = O.quantize_rows(x)
    assert s.view(np.uint16)[0, 0] == 0 and np.all(c == 0)
    assert np.all(O.dequantize(c, s, b) == v)


def test_affine_ladder_encodes_to_its_own_indices():
    for bias, step in [(0.0, 1.0), (-4.0, 0.5), (0.25, 0.0625), (-30.0, 4.0)]:
        ladder = bias + step * np.arange(16, dtype=np.float32)
        x = np.tile(ladder, 4)[None, :]
        assert np.array_equal(bf16(x), x)
        c, s, b = O.quantize_rows(x)
        assert float(s[0, 0]) == step and float(b[0, 0]) == bias
        assert np.array_equal(c[0], np.tile(np.arange(16), 4))
        assert np.array_equal(O.dequantize(c, s, b), x.astype(np.float64))


def test_min_is_code0_max_is_code15_and_codes_are_monotone():
    x = bf16(synth.rng(11, 0).standard_normal((32, 256), dtype=np.float32) * 3)
    c, s, b = O.quantize_rows(x)
    xg, cg = x.reshape(32, 4, 64), c.reshape(32, 4, 64)
    for r in range(32):
        for gi in range(4):
            assert cg[r, gi, xg[r, gi].argmin()] == 0
            assert cg[r, gi, xg[r, gi].argmax()] == 15
            order = np.argsort(xg[r, gi], kind="stable")
            assert np.all(np.diff(cg[r, gi][order].astype(int)) >= 0)


def test_groups_are_independent_and_along_head_dim():
    x = bf16(synth.rng(12, 0).standard_normal((3, 128), dtype=np.float32))
    c, s, b = O.quantize_rows(x)
    y = x.copy()
    y[:, 64:] *= 4.0                           # touching group 1 must not move group 0
    c2, s2, b2 = O.quantize_rows(y)
    assert np.array_equal(c[:, :64], c2[:, :64]) and np.array_equal(s[:, 0], s2[:, 0])
    assert not np.array_equal(s[:, 1], s2[:, 1])
