"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Packed codes, scales and biases must be bit-exact.  Attention outputs (float32) must satisfy
both  max |gpu - oracle| <= 2e-3  and, per output row, max_d |gpu - oracle| <= 1e-2 * max_d |oracle|
against the float64 oracle evaluated on the same dequantized values.
"""
import math

import numpy as np
import pytest
import torch

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth

pytestmark = pytest.mark.gpu

ATOL, RTOL_ROW = 2e-3, 1e-2


@pytest.fixture(scope="module")
def H():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_04428_b200 import harness
    return harness


def f32(bits):
    return synth.bf16_bits_to_f32(bits)


def assert_attention_close(gpu, ref, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    assert np.all(np.isfinite(gpu)), what
    err = np.abs(gpu - ref)
    assert err.max() <= ATOL, f"{what}: max abs err {err.max():.3e}"
    row_err = err.reshape(-1, ref.shape[-1]).max(axis=1)
    row_mag = np.abs(ref).reshape(-1, ref.shape[-1]).max(axis=1)
    bad = row_err > RTOL_ROW * row_mag + 1e-30
    assert not bad.any(), f"{what}: row-relative err {np.max(row_err / (row_mag + 1e-30)):.3e}"


def assert_lse_close(gpu, ref, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    fin = np.isfinite(ref)
    assert np.array_equal(np.isneginf(gpu), np.isneginf(ref)), what
    assert np.max(np.abs(gpu[fin] - ref[fin]), initial=0.0) <= 2e-3, what


class Pair:
    """The same cache on both sides: an oracle pool and a device pool behind one block table."""

    def __init__(self, H, spec_args, lens, seed, spare_blocks=3, extra_tokens=0, gain=1.0, outlier_frac=0.0,
                 exact_products=False, sb_dtype=0):
        L, Hq, Hkv, D, Dv, alias = spec_args
        self.H, self.lens, self.seed, self.gain, self.outlier_frac = H, list(lens), seed, gain, outlier_frac
        self.ospec = O.Spec(L, Hq, Hkv, D, Dv, alias, sb_dtype=sb_dtype)
        need = sum(-(-(n + extra_tokens) // 256) for n in lens)
        self.n_blocks = need + spare_blocks
        self.tabs = synth.block_tables(seed, 99, lens, self.n_blocks, extra_tokens=extra_tokens)
        self.opool = O.Pool(self.ospec, self.n_blocks, fill=0xFFFFFFFF)
        self.dc = H.DeviceCache(L, Hq, Hkv, D, Dv, alias, self.n_blocks, self.tabs, exact_products=exact_products,
                                sb_dtype=sb_dtype)

    def kv(self, layer, agent, n):
        s = self.ospec
        ko = vo = None
        if self.outlier_frac > 0:      # the recipe of the Llama-shaped configuration: a few channels carry 8x the values
            ko = synth.outlier_channels(self.seed, 100 + layer, s.n_kv_heads, s.d_qk, self.outlier_frac)
            vo = synth.outlier_channels(self.seed, 200 + layer, s.n_kv_heads, s.d_v, self.outlier_frac)
        k = synth.kv_bf16(self.seed, 1000 * layer + 10 * agent + 1, n, s.n_kv_heads, s.d_qk, ko)
        v = None if s.v_aliases_k else synth.kv_bf16(self.seed, 1000 * layer + 10 * agent + 2, n, s.n_kv_heads, s.d_v, vo)
        if self.gain != 1.0:
            k = synth.f32_to_bf16_bits(f32(k) * np.float32(self.gain))
            v = None if v is None else synth.f32_to_bf16_bits(f32(v) * np.float32(self.gain))
        return k, v

    def fill(self, chunks=None):
        """Append every agent's tokens on both sides, in the given chunk pattern (default: all at once)."""
        s = self.ospec
        for l in range(s.n_layers):
            data = [self.kv(l, a, n) for a, n in enumerate(self.lens)]
            done = [0] * len(self.lens)
            pattern = chunks or [max(self.lens)]
            for c in pattern:
                take = [min(c, n - d) for n, d in zip(self.lens, done)]
                offs = np.concatenate([[0], np.cumsum(take)]).astype(np.int32)
                if offs[-1] == 0:
                    continue
                kb = np.concatenate([data[a][0][done[a]:done[a] + take[a]] for a in range(len(take))])
                vb = None if s.v_aliases_k else np.concatenate(
                    [data[a][1][done[a]:done[a] + take[a]] for a in range(len(take))])
                O.quantize_append(self.opool, l, self.tabs, done, offs, f32(kb), None if vb is None else f32(vb))
                self.dc.append(l, done, offs, kb, vb)
                done = [d + t for d, t in zip(done, take)]
            assert done == self.lens
        return self

    def q(self, stream, n):
        return synth.normal_bf16(self.seed, stream, (n, self.ospec.n_q_heads, self.ospec.d_qk))

    def check_packed_equal(self):
        for a, n in enumerate(self.lens):
            ref = O.pack(self.opool, self.tabs[a], n)
            got = self.dc.pack(a, n).cpu().numpy()
            assert got.size == ref.size
            assert np.array_equal(got, ref), f"packed bytes differ for agent {a}"
        assert self.dc.read_flags() == 0


SPECS = {
    "gqa64": (2, 4, 2, 64, 64, False),
    "gqa128": (2, 8, 2, 128, 128, False),
    "gqa256": (1, 4, 2, 256, 256, False),
    "mla": (1, 16, 1, 576, 512, True),
    "asym": (1, 4, 4, 192, 128, False),
}


# ---- quantize-append and pack: bit-exact -------------------------------------------------------
@pytest.mark.parametrize("name", list(SPECS))
def test_quantize_append_and_pack_bit_exact(H, name):
    p = Pair(H, SPECS[name], [300, 17, 256], seed=21)
    p.fill(chunks=[5, 1, 2, 40, 1, 300])          # ragged starts: partial octets are read-modify-written
    p.check_packed_equal()


def test_quantize_append_adversarial_values_bit_exact(H):
    p = Pair(H, SPECS["gqa128"], [64], seed=22)
    s = p.ospec
    g = synth.rng(22, 5)
    x = g.standard_normal((64, s.n_kv_heads, s.d_qk), dtype=np.float32)
    x[1] *= 100.0
    x[2] = 1000.0 + 0.01 * x[2]
    x[3, :, :64] = 3.0
    x[4] *= 1e-6
    x[5, 0, 5] = 65280.0
    x[5, 0, 6] = -65280.0
    x[6] = 0.0
    x[7, :, 0] = -0.0
    x[8] *= 1e-7                                   # bias/scale in the binary16 subnormal range
    x[9] = np.round(x[9] * 2) / 2                  # many exact ties
    kb = synth.f32_to_bf16_bits(x)
    vb = synth.f32_to_bf16_bits(x[::-1].copy())
    for l in range(s.n_layers):
        O.quantize_append(p.opool, l, p.tabs, [0], [0, 64], f32(kb), f32(vb))
        p.dc.append(l, [0], [0, 64], kb, vb)
    p.check_packed_equal()


def test_unpack_then_pack_is_identity_and_attention_is_unchanged(H):
    p = Pair(H, SPECS["gqa128"], [700, 130], seed=23).fill()
    q = p.q(7, 2)
    out0, _ = p.dc.decode(1, p.lens, 0, q, 0.1)
    bufs = [p.dc.pack(a, n) for a, n in enumerate(p.lens)]
    # restore into other physical blocks of a fresh pool
    tabs2 = synth.block_tables(777, 1, p.lens, p.n_blocks + 5)
    assert not np.array_equal(tabs2[:, :1], p.tabs[:, :1]) or True
    dc2 = H.DeviceCache(*SPECS["gqa128"], p.n_blocks + 5, tabs2)
    for a, n in enumerate(p.lens):
        dc2.unpack(a, n, bufs[a])
        assert torch.equal(dc2.pack(a, n), bufs[a])
        assert np.array_equal(bufs[a].cpu().numpy(), O.pack(p.opool, p.tabs[a], n))
    out1, _ = dc2.decode(1, p.lens, 0, q, 0.1)
    assert torch.allclose(out0, out1, rtol=0, atol=1e-5)     # same bytes in other blocks; summation order may differ
    assert dc2.read_flags() == 0


def test_unpack_from_oracle_bytes_feeds_attention(H):
    """The device cache is filled ONLY from oracle-packed bytes: attention parity independent of the GPU quantizer."""
    p = Pair(H, SPECS["gqa64"], [515, 100], seed=24)
    s = p.ospec
    for l in range(s.n_layers):
        for a, n in enumerate(p.lens):
            k, v = p.kv(l, a, n)
            O.quantize_append(p.opool, l, p.tabs[a:a + 1], [0], [0, n], f32(k), f32(v))
    for a, n in enumerate(p.lens):
        p.dc.unpack(a, n, O.pack(p.opool, p.tabs[a], n))
    q = p.q(7, 2)
    for l in range(s.n_layers):
        ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, p.lens, 0, f32(q), 0.2)
        out, lse = p.dc.decode(l, p.lens, 0, q, 0.2)
        assert_attention_close(out.cpu().numpy(), ref, f"layer {l}")
        assert_lse_close(lse.cpu().numpy(), lse_ref)


class TiePair(Pair):
    """Keys and values whose quotients (x - bias) / scale sit exactly on, or one bf16 step beside, the rounding
    boundaries k + 1/2: min 0 and max 15 * 2^e per group, everything else (k + 1/2) * 2^e or its neighbours."""

    def kv(self, layer, agent, n):
        s = self.ospec
        rs = np.random.default_rng(1000 * layer + agent)

        def make(d):
            e = rs.integers(-6, 3, size=(n, s.n_kv_heads, d // 64, 1)).astype(np.float32)
            step = np.float32(2.0) ** e
            k = rs.integers(0, 15, size=(n, s.n_kv_heads, d // 64, 64)).astype(np.float32) + np.float32(0.5)
            x = k * step
            bits = synth.f32_to_bf16_bits(x.astype(np.float32))
            nudge = rs.integers(-1, 2, size=bits.shape).astype(np.int32)            # -1, 0, +1 bf16 ulp
            bits = (bits.astype(np.int32) + nudge).astype(np.uint16)
            x = f32(bits)
            x[..., 0] = 0.0
            x[..., 1] = (np.float32(15.0) * step)[..., 0]
            return synth.f32_to_bf16_bits(x.reshape(n, s.n_kv_heads, d).astype(np.float32))

        return make(s.d_qk), (None if s.v_aliases_k else make(s.d_v))


def test_quantizer_is_bit_exact_on_rounding_boundaries(H):
    """Every code decided at, or a hair beside, a tie: the reciprocal-and-correct quotient must fall back to the
    division exactly where it matters."""
    p = TiePair(H, SPECS["gqa128"], [300, 70], seed=23).fill(chunks=[3, 64, 300])
    p.check_packed_equal()
    p2 = TiePair(H, SPECS["mla"], [130], seed=24).fill()
    p2.check_packed_equal()


# ---- decode attention ---------------------------------------------------------------------------
def test_config1_tiny_decode_append_and_roundtrip(H):
    w = synth.workload(0)
    spec_args = (w.n_layers, w.n_q_heads, w.n_kv_heads, w.d_qk, w.d_v, w.v_aliases_k)
    p = Pair(H, spec_args, w.lens, seed=w.seed, spare_blocks=16 - 7, extra_tokens=1).fill()
    assert p.n_blocks == 16
    q = p.q(7, 2)
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, w.lens, 0, f32(q), w.softmax_scale)
    out, lse = p.dc.decode(0, w.lens, 0, q, w.softmax_scale)
    assert_attention_close(out.cpu().numpy(), ref, "before append")
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    # append one new token per agent, attend again (lengths 1001 / 701)
    kn = synth.kv_bf16(w.seed, 501, 2, w.n_kv_heads, w.d_qk)
    vn = synth.kv_bf16(w.seed, 502, 2, w.n_kv_heads, w.d_v)
    O.quantize_append(p.opool, 0, p.tabs, w.lens, [0, 1, 2], f32(kn), f32(vn))
    p.dc.append(0, w.lens, [0, 1, 2], kn, vn)
    lens1 = [n + 1 for n in w.lens]
    q1 = p.q(8, 2)
    ref1, _ = O.decode_attention(p.opool, 0, p.tabs, lens1, 0, f32(q1), w.softmax_scale)
    out1, _ = p.dc.decode(0, lens1, 0, q1, w.softmax_scale)
    assert_attention_close(out1.cpu().numpy(), ref1, "after append")
    p.lens = lens1
    p.check_packed_equal()


@pytest.mark.parametrize("name,lens,window", [
    ("gqa64", [20, 9, 262], 0),
    ("gqa64", [300, 17, 262], 12),
    ("gqa128", [1000, 700, 1, 255, 256, 257], 0),
    ("gqa128", [1000, 700, 33], 300),
    ("gqa256", [1500, 40], 0),
    ("gqa256", [1500, 1100], 1024),
    ("mla", [600, 70], 0),
    ("asym", [400, 300], 0),
    ("asym", [400, 300], 100),
    ("asym", [3000, 1, 31, 32, 33, 255, 256, 257, 0], 0),
])
def test_decode_matches_oracle(H, name, lens, window):
    p = Pair(H, SPECS[name], lens, seed=31).fill()
    s = p.ospec
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(s.d_qk if name != "mla" else 192)
    for l in range(s.n_layers):
        ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, lens, window, f32(q), scale)
        out, lse = p.dc.decode(l, lens, window, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"{name} layer {l}")
        assert_lse_close(lse.cpu().numpy(), lse_ref, name)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("spec_args,lens,window", [
    ((1, 16, 8, 256, 256, False), [30000, 9000], 0),       # ~66 chunks per CTA through a 20-slot ring
    ((1, 32, 8, 128, 128, False), [40000, 23000], 0),      # ~106 chunks per CTA through a 32-slot ring
    ((1, 16, 8, 256, 256, False), [30000, 9000], 1024),
    ((1, 16, 16, 192, 128, False), [20000, 5000], 0),      # d_qk 192 / d_v 128, one query head per KV head
])
def test_decode_long_contexts_wrap_the_ring(H, spec_args, lens, window):
    """Every CTA streams several times its shared-memory ring: slot reuse, ragged split and merge across many CTAs."""
    p = Pair(H, spec_args, lens, seed=37).fill()
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(spec_args[3])
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, window, f32(q), scale)
    out, lse = p.dc.decode(0, lens, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    # warps claim chunks dynamically, so the float32 summation order (not the result) varies from run to run
    out2, _ = p.dc.decode(0, lens, window, q, scale)
    assert torch.allclose(out, out2, rtol=0, atol=1e-5)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("spec_args,n_agents,max_len,window,fused", [
    ((1, 8, 2, 128, 128, False), 300, 200, 0, False),      # hundreds of short pairs: many segments per CTA
    ((1, 8, 2, 128, 128, False), 300, 200, 0, True),
    ((1, 4, 2, 256, 256, False), 150, 300, 64, True),
    ((1, 4, 4, 192, 128, False), 120, 150, 0, True),
    ((1, 8, 2, 128, 128, False), 40, 2500, 0, True),       # a few segments per CTA, pairs split over two or three CTAs
])
def test_decode_many_agents_many_segments_per_cta(H, spec_args, n_agents, max_len, window, fused):
    """Every CTA walks several (agent, KV head) segments: deposit buffers and query buffers are reused, segment
    epilogues run in the stream (by a consumer warp or, at d = 128, by the planner warp once all chunks are issued),
    pairs that straddle CTAs go through records and tickets.  Twice in a row on one workspace."""
    g = synth.rng(53, n_agents)
    lens = [int(x) for x in g.integers(1, max_len + 1, size=n_agents)]
    lens[3] = 0
    p = Pair(H, spec_args, lens, seed=53, extra_tokens=1, spare_blocks=2).fill()
    s = p.ospec
    scale = 1.0 / math.sqrt(s.d_qk)
    q = p.q(7, n_agents)
    if fused:
        kb = synth.kv_bf16(53, 500, n_agents, s.n_kv_heads, s.d_qk)
        vb = synth.kv_bf16(53, 600, n_agents, s.n_kv_heads, s.d_v)
        live = [a for a in range(n_agents) if lens[a] > 0]
        offs = np.concatenate([[0], np.cumsum([1 if lens[a] > 0 else 0 for a in range(n_agents)])]).astype(np.int32)
        O.quantize_append(p.opool, 0, p.tabs, lens, offs, f32(kb[live]), f32(vb[live]))
        new_lens = [n + 1 if n > 0 else 0 for n in lens]
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, new_lens, window, f32(q), scale)
        out, lse = p.dc.append_decode(0, new_lens, window, kb, vb, q, scale)
        p.lens = new_lens
    else:
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, window, f32(q), scale)
        out, lse = p.dc.decode(0, lens, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    out2, lse2 = p.dc.decode(0, p.lens, window, q, scale)          # the workspace header was left at zero
    assert_attention_close(out2.cpu().numpy(), ref, "second call")
    assert p.dc.read_flags() == 0
    if fused:
        p.check_packed_equal()


def test_decode_shorter_lengths_than_cached_and_zero_length(H):
    p = Pair(H, SPECS["gqa128"], [600, 300, 50], seed=32).fill()
    q = p.q(7, 3)
    lens = [257, 0, 1]
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), 0.09)
    out, lse = p.dc.decode(0, lens, 0, q, 0.09)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    assert torch.all(out[1] == 0)
    # kv_len = 1: exactly the dequantized V row 0
    _, V = O.gather_dequant(p.opool, 0, p.tabs[2], 0, 1, 1)
    assert np.allclose(out[2, 7].cpu().numpy(), V[0], rtol=0, atol=1e-6)
    assert p.dc.read_flags() == 0


def test_batched_equals_per_agent_calls(H):
    p = Pair(H, SPECS["gqa128"], [1000, 700, 256], seed=33).fill()
    q = p.q(7, 3)
    out, lse = p.dc.decode(1, p.lens, 0, q, 0.1)
    qd = H.bf16_dev(q)
    for a in range(3):
        t, bt = p.dc.sub_batch(a, a + 1)
        o1, l1 = p.dc.decode(1, p.lens[a:a + 1], 0, qd[a:a + 1].contiguous(), 0.1, bt=bt)
        # the split schedule depends on the batch size, so equality is within tolerance, not bitwise
        assert_attention_close(o1[0].cpu().numpy(), out[a].cpu().numpy().astype(np.float64), f"agent {a}")


def test_one_hot_keys_select_one_value_row(H):
    spec_args = (1, 2, 1, 64, 64, False)
    p = Pair(H, spec_args, [40], seed=34)
    perm = synth.rng(34, 0).permutation(64)[:40]
    k = np.zeros((40, 1, 64), dtype=np.float32)
    k[np.arange(40), 0, perm] = 7.5
    kb = synth.f32_to_bf16_bits(k)
    vb = synth.kv_bf16(34, 1, 40, 1, 64)
    O.quantize_append(p.opool, 0, p.tabs, [0], [0, 40], f32(kb), f32(vb))
    p.dc.append(0, [0], [0, 40], kb, vb)
    _, Vd = O.gather_dequant(p.opool, 0, p.tabs[0], 0, 40, 0)
    for m in (0, 13, 39):
        q = np.zeros((1, 2, 64), dtype=np.float32)
        q[0, :, perm[m]] = 16.0
        out, lse = p.dc.decode(0, [40], 0, synth.f32_to_bf16_bits(q), 1.0)
        assert np.max(np.abs(out[0, 1].cpu().numpy() - Vd[m])) <= 1e-5
        assert abs(float(lse[0, 0]) - 120.0) < 1e-3


def test_outlier_channels_large_values(H):
    """Values up to ~8x3 sigma (the outlier-channel recipe) still meet the absolute bound."""
    p = Pair(H, SPECS["gqa128"], [900, 400], seed=35)
    s = p.ospec
    for l in range(s.n_layers):
        for a, n in enumerate(p.lens):
            ko = synth.outlier_channels(35, 100 + l, s.n_kv_heads, s.d_qk)
            vo = synth.outlier_channels(35, 200 + l, s.n_kv_heads, s.d_v)
            kb = synth.kv_bf16(35, 1000 * l + 10 * a + 1, n, s.n_kv_heads, s.d_qk, ko)
            vb = synth.kv_bf16(35, 1000 * l + 10 * a + 2, n, s.n_kv_heads, s.d_v, vo)
            O.quantize_append(p.opool, l, p.tabs[a:a + 1], [0], [0, n], f32(kb), f32(vb))
            t, bt = p.dc.sub_batch(a, a + 1)
            p.dc.append(l, [0], [0, n], kb, vb, bt=bt)
    p.check_packed_equal()
    q = p.q(7, 2)
    ref, _ = O.decode_attention(p.opool, 1, p.tabs, p.lens, 0, f32(q), 1 / math.sqrt(128))
    out, _ = p.dc.decode(1, p.lens, 0, q, 1 / math.sqrt(128))
    assert_attention_close(out.cpu().numpy(), ref)


def test_bf16_output_mode(H):
    """bf16 output = the float32 result rounded once (nearest even); the float32 result is checked against the oracle."""
    from paper_2603_04428_b200 import binding as B
    p = Pair(H, SPECS["gqa128"], [500, 300], seed=36).fill()
    q = p.q(7, 2)
    ref, _ = O.decode_attention(p.opool, 0, p.tabs, p.lens, 0, f32(q), 0.1)
    out32, _ = p.dc.decode(0, p.lens, 0, q, 0.1)
    assert_attention_close(out32.cpu().numpy(), ref)
    out, _ = p.dc.decode(0, p.lens, 0, q, 0.1, out_dtype=B.OUT_BF16)
    assert out.dtype == torch.bfloat16
    assert torch.equal(out, out32.to(torch.bfloat16))
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + ATOL)      # half a bf16 ulp + the float32 bound


@pytest.mark.parametrize("spec_args,lens,window", [
    ((1, 16, 1, 576, 512, True), [5000, 700, 0, 63, 64, 65], 0),     # many key shares per agent, an empty agent, block edges
    ((1, 16, 1, 576, 512, True), [9000, 300], 1000),                 # a window that starts inside a 64-key block
    ((2, 8, 1, 576, 512, True), [2100], 0),                          # fewer than 16 heads, two layers
])
@pytest.mark.parametrize("exact", [False, True], ids=["tile", "codes"])
def test_decode_mla_latent_tensor_memory_path(H, spec_args, lens, window, exact):
    """The MLA-latent decode kernels: one binary16 tile per 64 keys serves as key and as value operand; with
    exact_products the 4-bit codes themselves do."""
    from paper_2603_04428_b200 import binding as B
    p = Pair(H, spec_args, lens, seed=37, exact_products=exact).fill()
    s = p.ospec
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(192)
    for l in range(s.n_layers):
        ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, lens, window, f32(q), scale)
        out, lse = p.dc.decode(l, lens, window, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"layer {l}")
        assert_lse_close(lse.cpu().numpy(), lse_ref)
    out16, _ = p.dc.decode(0, lens, window, q, scale, out_dtype=B.OUT_BF16)
    out32, _ = p.dc.decode(0, lens, window, q, scale)
    assert torch.allclose(out16.float(), out32.to(torch.bfloat16).float(), atol=1e-5, rtol=2.0 ** -7)
    assert p.dc.read_flags() == 0
    # a block id outside the pool poisons that agent only
    if lens[0] > 256:
        tabs = p.tabs.copy()
        tabs[0, 1] = p.n_blocks + 3
        t = H.dev(tabs)
        bad, lse_bad = p.dc.decode(0, lens, window, q, scale, bt=B.batch(t))
        hit = window == 0 or lens[0] - window < 512
        if hit:
            assert p.dc.read_flags() & B.FLAG_BAD_BLOCK
            assert torch.all(bad[0] == 0) and torch.isneginf(lse_bad[0]).all()
        assert torch.allclose(bad[1:], out32[1:], atol=1e-5)
        p.dc.flags.zero_()
    # a length beyond the block table is reported, and that agent's rows are zero
    over = [p.tabs.shape[1] * 256 + 1] + list(lens[1:])
    bad, lse_bad = p.dc.decode(0, over, window, q, scale)
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    assert torch.all(bad[0] == 0) and torch.isneginf(lse_bad[0]).all()
    assert torch.allclose(bad[1:], out32[1:], atol=1e-5)
    p.dc.flags.zero_()


@pytest.mark.parametrize("name,lens,window", [
    ("gqa128", [1000, 700, 0, 255, 256, 257, 31, 32, 33], 0),      # block and chunk edges, an agent without a token
    ("gqa128", [1000, 700, 64], 300),
    ("gqa256", [1500, 41, 2049], 1024),
    ("mla", [1000, 700, 0, 63, 64, 65, 129, 31, 32, 33], 0),       # the latent cache: 64-key block and chunk edges
    ("mla", [2500, 300, 4000], 200),
    ("asym", [1000, 700, 0, 255, 256, 257, 31, 32, 33], 0),        # d_qk 192 / d_v 128: the per-head MLA cache
    ("asym", [600, 90], 100),
])
def test_update_and_fetch_in_one_launch(H, name, lens, window):
    """q4kv_append_decode_attention: same pool bytes as quantize-append, same attention as decode, step after step."""
    from paper_2603_04428_b200 import binding as B
    spec_args = SPECS[name]
    steps = 3
    p = Pair(H, spec_args, lens, seed=39, extra_tokens=steps).fill()
    s = p.ospec
    A = len(lens)
    cur = list(lens)
    scale = 1.0 / math.sqrt(s.d_qk)
    for step in range(steps):
        kb = synth.kv_bf16(39, 500 + step, A, s.n_kv_heads, s.d_qk)
        vb = synth.kv_bf16(39, 600 + step, A, s.n_kv_heads, s.d_v)
        q = p.q(70 + step, A)
        live = [a for a in range(A) if lens[a] > 0]          # an agent that starts empty stays out of the step
        new_lens = [n + 1 if lens[a] > 0 else 0 for a, n in enumerate(cur)]
        for l in range(s.n_layers):
            # oracle: append row a at position cur[a] for the live agents, then attend
            offs = np.concatenate([[0], np.cumsum([1 if a in live else 0 for a in range(A)])]).astype(np.int32)
            O.quantize_append(p.opool, l, p.tabs, cur, offs, f32(kb[live]), f32(vb[live]))
            ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, new_lens, window, f32(q), scale)
            out, lse = p.dc.append_decode(l, new_lens, window, kb, vb, q, scale)
            assert_attention_close(out.cpu().numpy(), ref, f"{name} step {step} layer {l}")
            assert_lse_close(lse.cpu().numpy(), lse_ref, name)
        cur = new_lens
    p.lens = cur
    p.check_packed_equal()                                     # the pool holds exactly what quantize-append writes
    assert p.dc.read_flags() == 0



# ---- decode: head-group sizes, routes and workspace reuse that the cases above do not reach ------
@pytest.mark.parametrize("spec_args,lens,window", [
    ((1, 2, 2, 128, 128, False), [700, 33, 1000], 0),        # one query head per KV head
    ((1, 6, 2, 128, 128, False), [700, 33, 1000], 0),        # three: the fourth score row is absent
    ((1, 6, 2, 128, 128, False), [700, 33, 1000], 200),
    ((1, 3, 1, 256, 256, False), [1500, 41], 0),
    ((1, 2, 2, 256, 256, False), [1500, 41], 1024),
    ((1, 16, 2, 128, 128, False), [700, 300], 0),            # eight: beyond the tensor-core kernel, shape-agnostic path
    ((1, 16, 2, 128, 128, False), [700, 300], 100),
])
def test_decode_query_heads_per_kv_head(H, spec_args, lens, window):
    p = Pair(H, spec_args, lens, seed=41).fill()
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(spec_args[3])
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, window, f32(q), scale)
    out = torch.full((len(lens), spec_args[1], spec_args[4]), float("nan"), device="cuda")
    out, lse = p.dc.decode(0, lens, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("window", [0, 150])
def test_decode_latent_cache_at_a_sharp_scale_takes_the_exact_kernel(H, window):
    """scale^2 * d_qk > 4 on the V-aliasing cache: routed to the kernel that keeps the values exact."""
    lens = [600, 70, 257]
    p = Pair(H, SPECS["mla"], lens, seed=42).fill()
    q = p.q(7, len(lens))
    scale = 0.1
    assert scale * scale * 576 > 4
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, window, f32(q), scale)
    out, lse = p.dc.decode(0, lens, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("lens,window,scale,exact", [
    ([1000, 700, 0, 63, 64, 65, 129, 31, 32, 33], 0, 0.1, False),       # a sharp scale: 64-key block and chunk edges
    ([2500, 300, 4000], 200, 1.0 / math.sqrt(192), True),               # exact products asked for, a window
    ([9000, 1], 0, 0.1, True),                                          # many blocks per key share
])
def test_latent_cache_update_and_fetch_on_the_codes(H, lens, window, scale, exact):
    """The latent-cache calls that may not round the cache (exact_products, or scale^2 * d_qk > 4) run on the kernel
    that multiplies the 4-bit codes: update-and-fetch and the two-call form, pool bytes as quantize-append writes
    them, and the result within the bound of the exact routes (2e-5 * M + 1e-5, M the largest dequantized magnitude)."""
    steps = 2
    p = Pair(H, SPECS["mla"], lens, seed=45, extra_tokens=steps, exact_products=exact).fill()
    s = p.ospec
    A = len(lens)
    cur = list(lens)
    live = [a for a in range(A) if lens[a] > 0]
    for step in range(steps):
        kb = synth.kv_bf16(45, 500 + step, A, s.n_kv_heads, s.d_qk)
        q = p.q(70 + step, A)
        new_lens = [n + 1 if lens[a] > 0 else 0 for a, n in enumerate(cur)]
        offs = np.concatenate([[0], np.cumsum([1 if a in live else 0 for a in range(A)])]).astype(np.int32)
        O.quantize_append(p.opool, 0, p.tabs, cur, offs, f32(kb[live]), None)
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, new_lens, window, f32(q), scale)
        out, lse = p.dc.append_decode(0, new_lens, window, kb, None, q, scale)
        p.lens = new_lens
        M = max_dequantized_magnitude(p, 0)
        for what, (o, ls) in (("one launch", (out, lse)), ("two calls", p.dc.decode(0, new_lens, window, q, scale))):
            assert_attention_close(o.cpu().numpy(), ref, f"{what}, step {step}")
            assert_lse_close(ls.cpu().numpy(), lse_ref, what)
            assert np.abs(o.cpu().numpy().astype(np.float64) - ref).max() <= 2e-5 * M + 1e-5, what
        cur = new_lens
    p.check_packed_equal()
    assert p.dc.read_flags() == 0


def max_dequantized_magnitude(p, layer):
    m = 0.0
    for a, n in enumerate(p.lens):
        if n == 0:
            continue
        K, V = O.gather_dequant(p.opool, layer, p.tabs[a], 0, n, 0)
        m = max(m, float(np.abs(K).max()), float(np.abs(V).max()))
    return m


def tile_kernel_bound(p, layer, q_bits, scale):
    """The bound include/q4kv.h states for the kernels that round every dequantized value once to binary16:
    2^-10 * M * (1 + softmax_scale * max_rows ||q||_1 * M), M the largest dequantized magnitude (value and probability
    roundings, plus what the rounded keys do to the softmax weights)."""
    M = max_dequantized_magnitude(p, layer)
    q1 = float(np.abs(f32(q_bits)).sum(axis=-1).max())
    return M, 2.0 ** -10 * M * (1.0 + scale * q1 * M)


@pytest.mark.parametrize("gain,outlier_frac", [(8.0, 0.0), (1.0, 0.01)])
def test_latent_decode_on_large_magnitude_caches(H, gain, outlier_frac):
    """A cache with a gain of 8, or with 1 % of the channels carrying 8x the values: with exact_products the usual
    bound holds; without it the binary16-tile kernel stays inside the bound the header states for it."""
    lens = [900, 40, 1]
    q_bits = None
    for exact in (True, False):
        p = Pair(H, SPECS["mla"], lens, seed=43, gain=gain, outlier_frac=outlier_frac, exact_products=exact).fill()
        q_bits = p.q(7, len(lens))
        scale = 1.0 / math.sqrt(192)
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q_bits), scale)
        out, lse = p.dc.decode(0, lens, 0, q_bits, scale)
        got = out.cpu().numpy().astype(np.float64)
        if exact:
            assert_attention_close(got, ref, "exact products")
            assert_lse_close(lse.cpu().numpy(), lse_ref)
        else:
            M, bound = tile_kernel_bound(p, 0, q_bits, scale)
            assert M >= 8.0
            assert np.abs(got - ref).max() <= bound
        assert p.dc.read_flags() == 0


def test_one_workspace_serves_growing_batches_and_every_kernel(H):
    """One workspace, allocated once for the largest call and zero-filled once: a latent-cache call, a d = 192 call
    (shape-agnostic kernel) and GQA calls of 2 agents and then of 10 agents x 8 KV heads (more pairs than arrival
    counters fit in 256 bytes) all run on it, each compared with the oracle, outputs pre-filled with NaN."""
    from paper_2603_04428_b200 import binding as B
    cases = [
        (SPECS["mla"], [600, 70], 1.0 / math.sqrt(192)),
        (SPECS["asym"], [400, 300], 1.0 / math.sqrt(192)),
        ((1, 32, 8, 128, 128, False), [700, 300], 1.0 / math.sqrt(128)),
        ((1, 32, 8, 128, 128, False), [700, 300, 260, 5000, 90, 1200, 64, 33, 2000, 513], 1.0 / math.sqrt(128)),
        ((1, 32, 8, 128, 128, False), [700, 300], 1.0 / math.sqrt(128)),
    ]
    pairs = [Pair(H, sa, lens, seed=44 + i).fill() for i, (sa, lens, _) in enumerate(cases)]
    need = max(B.q4kv_workspace_bytes(p.dc.spec, len(p.lens), p.dc.bt.max_blocks * 256, 0) for p in pairs)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    for rounds in range(2):
        for p, (sa, lens, scale) in zip(pairs, cases):
            q = p.q(7 + rounds, len(lens))
            ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), scale)
            out = torch.full((len(lens), sa[1], sa[4]), float("nan"), device="cuda")
            lse = torch.full((len(lens), sa[1]), float("nan"), device="cuda")
            B.q4kv_decode_attention(p.dc.spec, p.dc.pool, p.dc.n_blocks, 0, p.dc.bt, H.dev(np.asarray(lens, dtype=np.int32)),
                                    0, 0, H.bf16_dev(q), scale, out, B.OUT_F32, lse, ws, p.dc.flags)
            assert_attention_close(out.cpu().numpy(), ref, f"{sa} {len(lens)} agents")
            assert_lse_close(lse.cpu().numpy(), lse_ref)
            assert p.dc.read_flags() == 0
    assert int(ws[:B.WORKSPACE_HEADER_BYTES].max()) == 0          # every call left the arrival counters at zero


@pytest.mark.parametrize("name", ["gqa128", "mla", "asym"])
def test_length_beyond_the_stated_maximum_is_flagged_on_every_kernel(H, name):
    """max_kv_len is the caller's bound on every length: an agent above it gets zeros and Q4KV_FLAG_BAD_LENGTH,
    whichever kernel serves the spec; the other agents are unaffected."""
    from paper_2603_04428_b200 import binding as B
    lens = [900, 300]
    p = Pair(H, SPECS[name], lens, seed=45).fill()
    q = p.q(7, 2)
    scale = 1.0 / math.sqrt(192 if name == "mla" else p.ospec.d_qk)
    ref, _ = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), scale)
    out, lse = p.dc.decode(0, lens, 0, q, scale, max_kv_len=512)
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    assert torch.all(out[0] == 0) and torch.isneginf(lse[0]).all()
    assert_attention_close(out[1].cpu().numpy(), ref[1])
    p.dc.flags.zero_()



@pytest.mark.parametrize("spec_args,lens,windows,fused", [
    ((3, 8, 2, 128, 128, False), [1000, 700, 0, 33, 257], [0, 0, 0], False),
    ((4, 8, 2, 128, 128, False), [1000, 700, 64], [300, 0, 300, 0], True),        # window and global layers in one launch
    ((2, 4, 2, 256, 256, False), [1500, 41, 2049], [1024, 0], True),
    ((2, 16, 16, 192, 128, False), [700, 33, 300], [0, 0], True),     # the per-head MLA cache, 16 KV heads
])
def test_layer_batched_decode_equals_the_oracle_layer_by_layer(H, spec_args, lens, windows, fused):
    """q4kv_decode_attention_layers: all layers of a step in one launch (work list over layers x agents x KV heads),
    with and without the fused append, against the oracle layer by layer; the pool ends up with the appended rows."""
    from paper_2603_04428_b200 import binding as B
    L = spec_args[0]
    p = Pair(H, spec_args, lens, seed=71, extra_tokens=1).fill()
    s = p.ospec
    A = len(lens)
    scale = 1.0 / math.sqrt(s.d_qk)
    new_lens = [n + 1 if (fused and n > 0) else n for n in lens]
    q_all = np.stack([p.q(80 + l, A) for l in range(L)])
    kb = np.stack([synth.kv_bf16(71, 500 + l, A, s.n_kv_heads, s.d_qk) for l in range(L)])
    vb = np.stack([synth.kv_bf16(71, 600 + l, A, s.n_kv_heads, s.d_v) for l in range(L)])
    live = [a for a in range(A) if lens[a] > 0]
    refs, lses = [], []
    for l in range(L):
        if fused:
            offs = np.concatenate([[0], np.cumsum([1 if a in live else 0 for a in range(A)])]).astype(np.int32)
            O.quantize_append(p.opool, l, p.tabs, lens, offs, f32(kb[l][live]), f32(vb[l][live]))
        r, ls = O.decode_attention(p.opool, l, p.tabs, new_lens, windows[l], f32(q_all[l]), scale)
        refs.append(r); lses.append(ls)
    out = torch.full((L, A, s.n_q_heads, s.d_v), float("nan"), device="cuda")
    lse = torch.full((L, A, s.n_q_heads), float("nan"), device="cuda")
    need = B.q4kv_workspace_bytes_layers(p.dc.spec, A, p.dc.bt.max_blocks * 256, L)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    lens_d = H.dev(np.asarray(new_lens, dtype=np.int32))
    for rounds in range(2 if not fused else 1):                 # the workspace header is left at zero: a second call works
        B.q4kv_decode_attention_layers(p.dc.spec, p.dc.pool, p.dc.n_blocks, 0, L, p.dc.bt, lens_d, 0, windows,
                                       H.bf16_dev(kb) if fused else None, H.bf16_dev(vb) if fused else None,
                                       H.bf16_dev(q_all), scale, out, B.OUT_F32, lse, ws, p.dc.flags)
        for l in range(L):
            assert_attention_close(out[l].cpu().numpy(), refs[l], f"layer {l}")
            assert_lse_close(lse[l].cpu().numpy(), lses[l])
    assert int(ws[:B.WORKSPACE_HEADER_BYTES].max()) == 0
    p.lens = new_lens
    p.check_packed_equal()


# ---- prefill attention --------------------------------------------------------------------------
@pytest.mark.parametrize("name,prefix,chunk,window", [
    ("gqa64", [300, 70], 40, 0),
    ("gqa64", [300, 70], 40, 50),
    ("gqa128", [512, 200], 130, 0),
    ("gqa256", [256, 10], 70, 128),
    ("mla", [200], 33, 0),
    ("asym", [300, 70], 40, 0),
    ("asym", [300, 70], 40, 50),
])
def test_prefill_matches_oracle_and_chunking_is_invisible(H, name, prefix, chunk, window):
    lens = [n + chunk for n in prefix]
    p = Pair(H, SPECS[name], lens, seed=41).fill(chunks=[max(prefix), chunk])
    s = p.ospec
    A = len(lens)
    q_offs = [chunk * a for a in range(A + 1)]
    q = p.q(7, chunk * A)
    scale = 1.0 / math.sqrt(s.d_qk)
    ref, lse_ref = O.prefill_attention(p.opool, 0, p.tabs, lens, q_offs, window, f32(q), scale)
    out, lse = p.dc.prefill(0, lens, q_offs, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref, name)
    assert_lse_close(lse.cpu().numpy(), lse_ref, name)
    # second half alone, as its own chunk over the same cache: same rows
    h = chunk // 2
    rows = np.concatenate([np.arange(chunk * a + h, chunk * (a + 1)) for a in range(A)])
    q2 = q[rows]
    offs2 = [(chunk - h) * a for a in range(A + 1)]
    out2, _ = p.dc.prefill(0, lens, offs2, window, q2, scale)
    assert_attention_close(out2.cpu().numpy(), ref[rows], name + " second chunk")
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("spec_args,prefix,chunks,window", [
    ((1, 8, 2, 128, 128, False), [700, 0, 33], [200, 77, 130], 0),       # several 64-query tiles, an empty prefix
    ((1, 8, 2, 128, 128, False), [700, 300], [200, 150], 96),            # sliding window across chunk edges
    ((1, 4, 4, 128, 128, False), [2500], [300], 0),                      # MHA (one query head per KV head)
    ((2, 6, 2, 128, 128, False), [100, 40], [65, 1], 0),                 # three query heads per KV head, a 1-token phase
    ((1, 8, 4, 256, 256, False), [700, 0, 33], [150, 77, 130], 0),       # d = 256, two query heads per KV head
    ((1, 8, 4, 256, 256, False), [1400, 300], [200, 150], 512),          # d = 256 under a sliding window
    ((1, 4, 4, 256, 256, False), [900], [131], 0),                       # d = 256, one query head per KV head
    ((1, 8, 2, 256, 256, False), [300, 40], [65, 1], 100),               # d = 256, four query heads per KV head
    ((1, 6, 2, 256, 256, False), [300, 40], [65, 33], 0),                # d = 256, three query heads per KV head
])
def test_prefill_tensor_core_path_ragged(H, spec_args, prefix, chunks, window):
    """Ragged phases through the tensor-core prefill kernels (d = 128 and d = 256): every row against the oracle."""
    lens = [p0 + c for p0, c in zip(prefix, chunks)]
    p = Pair(H, spec_args, lens, seed=43).fill()
    s = p.ospec
    q_offs = np.concatenate([[0], np.cumsum(chunks)]).astype(np.int32)
    q = p.q(7, int(q_offs[-1]))
    scale = 1.0 / math.sqrt(s.d_qk)
    for l in range(s.n_layers):
        ref, lse_ref = O.prefill_attention(p.opool, l, p.tabs, lens, q_offs, window, f32(q), scale)
        out, lse = p.dc.prefill(l, lens, q_offs, window, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"layer {l}")
        assert_lse_close(lse.cpu().numpy(), lse_ref)
    # row i of the phase equals a decode call at kv_len = prefix + i + 1
    a, i = 0, chunks[0] // 2
    row = int(q_offs[a]) + i
    ref_d, _ = O.decode_attention(p.opool, 0, p.tabs[a:a + 1], [prefix[a] + i + 1], window, f32(q[row:row + 1]), scale)
    out0, _ = p.dc.prefill(0, lens, q_offs, window, q, scale)
    assert_attention_close(out0[row:row + 1].cpu().numpy(), ref_d)
    assert p.dc.read_flags() == 0


def test_interleaved_512_token_chunks_and_decoding_agents_in_one_batch(H):
    """The scheduler's pattern of Section 3.4: prompts are prefilled in chunks of at most 512 tokens, the chunks of
    different agents interleaved step by step, while another agent decodes one token per step -- every step is ONE
    append call and ONE attention call over a ragged batch (chunk lengths 512, 188, 1 ...).  Every row must equal the
    oracle's one-shot prefill of the whole prompt (the chunking is invisible), and the cache bytes its append."""
    spec_args = (1, 8, 2, 128, 128, False)
    prompts = [1700, 700, 0]                     # agent 2 has a cached context and decodes
    cached = [0, 300, 900]                       # tokens already in the cache when the schedule starts
    steps = 3
    total = [cached[a] + (prompts[a] if prompts[a] else steps) for a in range(3)]
    p = Pair(H, spec_args, total, seed=47)
    s = p.ospec
    data = [p.kv(0, a, total[a]) for a in range(3)]
    qs = [p.q(20 + a, total[a] - cached[a]) for a in range(3)]       # one query row per new token
    scale = 1.0 / math.sqrt(s.d_qk)
    # the cached contexts
    for a in range(3):
        if cached[a]:
            O.quantize_append(p.opool, 0, p.tabs[a:a + 1], [0], [0, cached[a]], f32(data[a][0][:cached[a]]), f32(data[a][1][:cached[a]]))
    p.dc.append(0, [0, 0, 0], np.concatenate([[0], np.cumsum(cached)]).astype(np.int32),
                np.concatenate([data[a][0][:cached[a]] for a in range(3)]), np.concatenate([data[a][1][:cached[a]] for a in range(3)]))
    # oracle, one shot: each agent's new tokens as a single phase
    for a in range(3):
        O.quantize_append(p.opool, 0, p.tabs[a:a + 1], [cached[a]], [0, total[a] - cached[a]],
                          f32(data[a][0][cached[a]:]), f32(data[a][1][cached[a]:]))
    refs = []
    for a in range(3):
        n_new = total[a] - cached[a]
        r, _ = O.prefill_attention(p.opool, 0, p.tabs[a:a + 1], [total[a]], [0, n_new], 0, f32(qs[a]), scale)
        refs.append(r)
    # the schedule: step t takes up to 512 prompt tokens of every prefilling agent and one token of the decoding one
    done = [0, 0, 0]
    for t in range(steps):
        take = [min(512, prompts[a] - done[a]) if prompts[a] else 1 for a in range(3)]
        assert any(take)
        pos = [cached[a] + done[a] for a in range(3)]
        offs = np.concatenate([[0], np.cumsum(take)]).astype(np.int32)
        kb = np.concatenate([data[a][0][pos[a]:pos[a] + take[a]] for a in range(3)])
        vb = np.concatenate([data[a][1][pos[a]:pos[a] + take[a]] for a in range(3)])
        qb = np.concatenate([qs[a][done[a]:done[a] + take[a]] for a in range(3)])
        p.dc.append(0, pos, offs, kb, vb)
        lens = [pos[a] + take[a] for a in range(3)]
        out, _ = p.dc.prefill(0, lens, offs, 0, qb, scale)
        got = out.cpu().numpy()
        for a in range(3):
            if take[a]:
                assert_attention_close(got[offs[a]:offs[a + 1]], refs[a][done[a]:done[a] + take[a]], f"step {t} agent {a}")
        done = [done[a] + take[a] for a in range(3)]
    assert done == [512 * steps, 700, steps]
    # agent 0 still has 164 tokens left: a fourth step on its own
    rest = prompts[0] - done[0]
    if rest:
        pos0 = cached[0] + done[0]
        p.dc.append(0, [pos0], [0, rest], data[0][0][pos0:], data[0][1][pos0:], bt=p.dc.sub_batch(0, 1)[1])
        t0, b0 = p.dc.sub_batch(0, 1)
        out, _ = p.dc.prefill(0, [total[0]], [0, rest], 0, qs[0][done[0]:], scale, bt=b0)
        assert_attention_close(out.cpu().numpy(), refs[0][done[0]:], "agent 0 tail")
    p.lens = total
    p.check_packed_equal()


class QuietStartPair(Pair):
    """The first 300 keys of every agent are tiny, so every row's running maximum jumps far when the walk leaves them."""

    def kv(self, layer, agent, n):
        k, v = super().kv(layer, agent, n)
        kf = f32(k).copy()
        kf[:300] *= np.float32(0.02)
        return synth.f32_to_bf16_bits(kf), v


@pytest.mark.parametrize("spec_args,prefix,chunks,window,scale_mul", [
    ((1, 4, 2, 128, 128, False), [900, 5], [140, 70], 0, 1.0),           # two query heads per KV head: 64-query tiles
    ((1, 8, 2, 128, 128, False), [3000], [200], 700, 1.0),               # the window starts many 64-key blocks in
    ((1, 8, 2, 128, 128, False), [1500, 64], [129, 64], 0, 2.0),         # the row maximum jumps by more than 2^8, late
    ((1, 8, 2, 128, 128, False), [1500, 64], [129, 64], 0, 8.0),         # a sharp scale is routed to the exact-code kernel
    ((1, 6, 2, 128, 128, False), [700, 30], [100, 64], 0, 1.0),          # three query heads per KV head: exact-code kernel
    ((1, 4, 4, 128, 128, False), [0], [257], 0, 1.0),                    # no prefix at all: purely causal
    ((1, 4, 2, 256, 256, False), [900, 5], [140, 70], 0, 1.0),           # d = 256 (one tile per CTA, two score buffers)
    ((1, 8, 2, 256, 256, False), [3000], [200], 700, 1.0),               # d = 256, four heads per KV head, a window
    ((1, 8, 2, 256, 256, False), [1500, 64], [129, 64], 0, 2.0),         # d = 256, the row maximum jumps by more than 2^8
    ((1, 4, 4, 256, 256, False), [0], [257], 0, 1.0),                    # d = 256, no prefix, one head per KV head
    ((1, 2, 1, 256, 256, False), [6000, 1], [300, 1], 0, 1.0),           # d = 256, ~100 blocks through the two-stage rings; one key
    ((1, 4, 4, 192, 128, False), [900, 5], [140, 70], 0, 1.0),           # d_qk 192 / d_v 128 (the same one-tile kernel), one head per KV head
    ((1, 8, 2, 192, 128, False), [3000], [200], 700, 1.0),               # 192 / 128, four heads per KV head, a window
    ((1, 4, 2, 192, 128, False), [1500, 64], [129, 64], 0, 2.0),         # 192 / 128, the row maximum jumps by more than 2^8
    ((1, 16, 16, 192, 128, False), [0, 33, 5000], [257, 31, 100], 0, 1.0),   # 192 / 128, sixteen KV heads, no prefix, a long prefix
    ((1, 2, 2, 256, 256, False), [30000], [64], 0, 1.0),                 # d = 256: 470 blocks, every ring wraps hundreds of times
    ((1, 2, 2, 192, 128, False), [20000, 300], [100, 10], 0, 1.0),       # 192 / 128: 314 blocks
    ((1, 4, 1, 128, 128, False), [30000], [64], 0, 1.0),                 # d = 128 (two tiles, one of them empty): 470 blocks
])
def test_prefill_tcgen05_path(H, spec_args, prefix, chunks, window, scale_mul):
    """The tensor-memory prefill kernel: tile shapes for 1, 2 and 4 heads per KV head, key ranges that start
    inside the cache, wrap the shared-memory stages many times, and scores whose maximum grows in steps both
    smaller and larger than the lazy-rescale threshold."""
    lens = [p0 + c for p0, c in zip(prefix, chunks)]
    p = QuietStartPair(H, spec_args, lens, seed=47).fill()
    s = p.ospec
    q_offs = np.concatenate([[0], np.cumsum(chunks)]).astype(np.int32)
    q = p.q(9, int(q_offs[-1]))
    scale = scale_mul / math.sqrt(s.d_qk)
    ref, lse_ref = O.prefill_attention(p.opool, 0, p.tabs, lens, q_offs, window, f32(q), scale)
    out, lse = p.dc.prefill(0, lens, q_offs, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    from paper_2603_04428_b200 import binding as B
    out16, _ = p.dc.prefill(0, lens, q_offs, window, q, scale, out_dtype=B.OUT_BF16)
    assert torch.allclose(out16.float(), out.to(torch.bfloat16).float(), atol=1e-5, rtol=2.0 ** -7)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("gain,outlier_frac", [(8.0, 0.0), (1.0, 0.01)])
@pytest.mark.parametrize("prefix,chunks", [([0, 40], [70, 30]), ([300], [64])])
@pytest.mark.parametrize("d", [128, 256, 192])
def test_prefill_on_large_magnitude_caches(H, gain, outlier_frac, prefix, chunks, d):
    """Rows that attend 1 to 64 keys of a cache with a gain of 8, or with 1 % of the channels carrying 8x the
    values, return value rows almost verbatim, so a single binary16 rounding of a dequantized value (half an ulp of
    2^-8 for magnitudes in [8, 16)) is visible.  With exact_products the usual bound holds; without it the
    binary16-tile kernel stays inside the bound the header states for it."""
    spec_args = (1, 8, 2, d, 128 if d == 192 else d, False)
    lens = [p0 + c for p0, c in zip(prefix, chunks)]
    q_offs = np.concatenate([[0], np.cumsum(chunks)]).astype(np.int32)
    scale = 1.0 / math.sqrt(d)
    for exact in (True, False):
        p = Pair(H, spec_args, lens, seed=48, gain=gain, outlier_frac=outlier_frac, exact_products=exact).fill()
        q = p.q(9, int(q_offs[-1]))
        ref, lse_ref = O.prefill_attention(p.opool, 0, p.tabs, lens, q_offs, 0, f32(q), scale)
        out, lse = p.dc.prefill(0, lens, q_offs, 0, q, scale)
        got = out.cpu().numpy().astype(np.float64)
        if exact:
            assert_attention_close(got, ref, "exact products")
            assert_lse_close(lse.cpu().numpy(), lse_ref)
        else:
            M, bound = tile_kernel_bound(p, 0, q, scale)
            assert M >= 8.0
            assert np.abs(got - ref).max() <= bound
        assert p.dc.read_flags() == 0


@pytest.mark.parametrize("d", [128, 256, 192])
def test_prefill_bad_block_and_bad_length(H, d):
    from paper_2603_04428_b200 import binding as B
    lens = [600, 200]
    p = Pair(H, (1, 8, 2, d, 128 if d == 192 else d, False), lens, seed=53).fill()
    q_offs = [0, 100, 180]
    q = p.q(7, 180)
    good, _ = p.dc.prefill(0, lens, q_offs, 0, q, 0.1)
    tabs = p.tabs.copy()
    tabs[0, 1] = -5
    t = H.dev(tabs)
    out, lse = p.dc.prefill(0, lens, q_offs, 0, q, 0.1, bt=B.batch(t))
    assert p.dc.read_flags() & B.FLAG_BAD_BLOCK
    assert torch.all(out[:100] == 0) and torch.equal(out[100:], good[100:])
    assert torch.all(torch.isneginf(lse[:100]))
    p.dc.flags.zero_()
    out, _ = p.dc.prefill(0, [50, 200], q_offs, 0, q, 0.1)          # more new tokens than cached tokens
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    assert torch.all(out[:100] == 0) and torch.equal(out[100:], good[100:])
    p.dc.flags.zero_()



def test_tensor_memory_prefill_and_latent_decode_repeat_bit_for_bit(H):
    """The kernels whose warps hand tiles to one another through mbarriers (tensor-memory prefill at d = 128 and 256,
    latent-cache decode on tiles and on codes) have a fixed order of arithmetic: sixty launches in a row on the same
    inputs return the same bits, which a missed hand-off (a tile read before it is complete) would not."""
    for spec_args, prefix, chunk in (((1, 8, 2, 128, 128, False), [1800, 300], 200),
                                     ((1, 8, 4, 256, 256, False), [1800, 300], 200),
                                     ((1, 8, 8, 192, 128, False), [1800, 300], 200)):
        lens = [n + chunk for n in prefix]
        p = Pair(H, spec_args, lens, seed=91).fill()
        q_offs = [0, chunk, 2 * chunk]
        q = H.bf16_dev(p.q(7, 2 * chunk))
        scale = 1.0 / math.sqrt(spec_args[3])
        first, lse0 = p.dc.prefill(0, lens, q_offs, 0, q, scale)
        for _ in range(60):
            out, lse = p.dc.prefill(0, lens, q_offs, 0, q, scale)
            assert torch.equal(out, first) and torch.equal(lse, lse0)
        assert p.dc.read_flags() == 0
    for exact in (False, True):
        lens = [5000, 700, 64]
        p = Pair(H, SPECS["mla"], lens, seed=92, exact_products=exact).fill()
        q = H.bf16_dev(p.q(7, len(lens)))
        first, lse0 = p.dc.decode(0, lens, 0, q, 1.0 / math.sqrt(192))
        for _ in range(60):
            out, lse = p.dc.decode(0, lens, 0, q, 1.0 / math.sqrt(192))
            assert torch.equal(out, first) and torch.equal(lse, lse0)
        assert p.dc.read_flags() == 0


# ---- persisted container and warm restore --------------------------------------------------------
@pytest.mark.parametrize("name,lens", [("gqa128", [700, 33]), ("mla", [300, 256]), ("asym", [17, 513])])
def test_saved_file_image_equals_the_oracles_and_restores_into_other_blocks(H, name, lens, tmp_path):
    """q4kv_save writes exactly the oracle's file image (canonical header + packed bytes); the image, written to a file
    and read back, is restored by q4kv_restore into another cache's blocks (chunked copies overlapping the scatter),
    after which that cache packs to the same bytes and attends to the same result."""
    p = Pair(H, SPECS[name], lens, seed=61).fill()
    s = p.ospec
    images = []
    for a, n in enumerate(lens):
        img = p.dc.save(a, n)
        ref = O.container(p.opool, p.tabs[a], n)
        assert img.numel() == ref.size and np.array_equal(img.numpy(), ref), f"agent {a}"
        f = tmp_path / f"agent{a}.safetensors"
        f.write_bytes(img.numpy().tobytes())
        images.append(f)
    # a second cache with other physical blocks
    p2 = Pair(H, SPECS[name], lens, seed=62)
    for a, n in enumerate(lens):
        raw = np.fromfile(images[a], dtype=np.uint8)
        img = torch.from_numpy(raw).pin_memory()
        for stage_layers in (1, 2):                                   # one staging half, then two
            assert p2.dc.restore(a, img, staging_layers=stage_layers) == n
            assert np.array_equal(p2.dc.pack(a, n).cpu().numpy(), O.pack(p.opool, p.tabs[a], n))
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(192 if name == "mla" else s.d_qk)
    ref, _ = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), scale)
    out, _ = p2.dc.decode(0, lens, 0, q, scale)
    assert_attention_close(out.cpu().numpy(), ref)
    assert p.dc.read_flags() == 0 and p2.dc.read_flags() == 0



@pytest.mark.parametrize("name,lens,T", [("gqa128", [300, 5, 0, 256, 33], 320), ("mla", [70, 513], 520), ("asym", [17, 290], 290)])
def test_dense_batch_extract_and_merge_match_the_oracle(H, name, lens, T):
    """The paper's merge / extract as a shim: a layer's caches as one left-padded dense batch, bytes equal to the
    oracle's, and merged back into other blocks (partly filled chunks keep their neighbours' slots) to the same cache."""
    from paper_2603_04428_b200 import binding as B
    p = Pair(H, SPECS[name], lens, seed=63).fill()
    s = p.ospec
    A = len(lens)
    lens_d = H.dev(np.asarray(lens, dtype=np.int32))
    nbytes = B.q4kv_dense_bytes(p.dc.spec, A, T)
    layer = s.n_layers - 1
    dense = torch.full((nbytes,), 0xAB, dtype=torch.uint8, device="cuda")
    B.q4kv_extract_dense(p.dc.spec, p.dc.pool, p.dc.n_blocks, layer, p.dc.bt, lens_d, T, dense, p.dc.flags)
    ref = O.extract_dense(p.opool, layer, p.tabs, lens, T)
    assert ref.size == nbytes and np.array_equal(dense.cpu().numpy(), ref)
    # merge into a cache that already holds other tokens: positions >= len keep what was there
    longer = [n + 40 for n in lens]
    p2 = Pair(H, SPECS[name], longer, seed=64).fill()
    B.q4kv_merge_dense(p2.dc.spec, p2.dc.pool, p2.dc.n_blocks, layer, p2.dc.bt, lens_d, T, dense, p2.dc.flags)
    O.merge_dense(p2.opool, layer, p2.tabs, lens, T, ref)
    p2.check_packed_equal()                                      # every layer, all longer[a] positions
    # a length beyond the dense row count is flagged and skipped
    bad = H.dev(np.asarray([T + 1] + lens[1:], dtype=np.int32))
    B.q4kv_extract_dense(p.dc.spec, p.dc.pool, p.dc.n_blocks, layer, p.dc.bt, bad, T, dense, p.dc.flags)
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    p.dc.flags.zero_()


# ---- anomalies are reported, not faulted on -----------------------------------------------------
def test_bad_block_id_and_bad_length_raise_flags_and_zero_output(H):
    from paper_2603_04428_b200 import binding as B
    p = Pair(H, SPECS["gqa64"], [300, 100], seed=51).fill()
    q = p.q(7, 2)
    good, _ = p.dc.decode(0, p.lens, 0, q, 0.1)
    tabs = p.tabs.copy()
    tabs[0, 1] = p.n_blocks + 7                     # outside the pool
    t = H.dev(tabs)
    out, _ = p.dc.decode(0, p.lens, 0, q, 0.1, bt=B.batch(t))
    assert p.dc.read_flags() & B.FLAG_BAD_BLOCK
    assert torch.all(out[0] == 0) and torch.equal(out[1], good[1])
    p.dc.flags.zero_()
    out, _ = p.dc.decode(0, [p.tabs.shape[1] * 256 + 1, 100], 0, q, 0.1)
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    assert torch.all(out[0] == 0) and torch.equal(out[1], good[1])
    p.dc.flags.zero_()
    out, _ = p.dc.decode(0, [-3, 100], 0, q, 0.1)
    assert p.dc.read_flags() & B.FLAG_BAD_LENGTH
    assert torch.all(out[0] == 0)


def test_host_side_rejections(H):
    from paper_2603_04428_b200 import binding as B
    p = Pair(H, SPECS["gqa64"], [100], seed=52).fill()
    bad = B.Spec.make(1, 4, 2, 96, 64)
    assert B.q4kv_pool_bytes(bad, 4) == 0
    with pytest.raises(B.Q4KVError) as e:
        B.q4kv_decode_attention(bad, p.dc.pool, p.n_blocks, 0, p.dc.bt, p.dc.tables, 0, 0, p.dc.pool, 0.1, p.dc.pool,
                                0, None, p.dc.pool, None)
    assert e.value.code == B.EUNSUPPORTED
    q = H.bf16_dev(p.q(7, 1))
    out = torch.empty((1, 4, 64), device="cuda")
    tiny = torch.empty(16, dtype=torch.uint8, device="cuda")
    lens = H.dev(np.array([100], dtype=np.int32))
    with pytest.raises(B.Q4KVError) as e:
        B.q4kv_decode_attention(p.dc.spec, p.dc.pool, p.n_blocks, 0, p.dc.bt, lens, 0, 0, q, 0.1, out, 0, None, tiny)
    assert e.value.code == B.EWORKSPACE
    with pytest.raises(B.Q4KVError) as e:
        B.q4kv_decode_attention(p.dc.spec, p.dc.pool, p.n_blocks, 5, p.dc.bt, lens, 0, 0, q, 0.1, out, 0, None, tiny)
    assert e.value.code == B.EINVAL
    dst = torch.empty(100, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.Q4KVError) as e:
        B.q4kv_pack(p.dc.spec, p.dc.pool, p.n_blocks, p.dc.tables[0], 100, dst)
    assert e.value.code == B.EWORKSPACE


# ---- the benchmark's own launches, at full size -------------------------------------------------
class WorkloadPair(Pair):
    """One layer of a benchmark configuration: its agents, lengths, head shapes and outlier channels."""

    def __init__(self, H, w, extra_tokens):
        super().__init__(H, (1, w.n_q_heads, w.n_kv_heads, w.d_qk, w.d_v, w.v_aliases_k), list(w.lens), seed=w.seed,
                         extra_tokens=extra_tokens)
        self.w = w
        self.ko = synth.outlier_channels(w.seed, 100, w.n_kv_heads, w.d_qk, w.outlier_frac) if w.outlier_frac else None
        self.vo = synth.outlier_channels(w.seed, 200, w.n_kv_heads, w.d_v, w.outlier_frac) if w.outlier_frac else None

    def kv(self, layer, agent, n):
        w = self.w
        k = synth.kv_bf16(w.seed, 10 * agent + 1, n, w.n_kv_heads, w.d_qk, outliers=self.ko)
        v = None if w.v_aliases_k else synth.kv_bf16(w.seed, 10 * agent + 2, n, w.n_kv_heads, w.d_v, outliers=self.vo)
        return k, v


@pytest.mark.parametrize("index", [1, 2, 3])
def test_full_size_decode_launches_match_the_oracle(H, index):
    """Configurations 2, 3 and 4 exactly as bench.py launches them, one layer: every agent, every head, every
    cached token (4096 x 5; ten ragged agents up to 32k tokens, window and global layer; 16384 x 4 MLA latents),
    the step's new token appended by the library, then every output row against the fp64 oracle."""
    w = synth.workload(index)
    p = WorkloadPair(H, w, extra_tokens=1).fill(chunks=[8192] * 4)
    s = p.ospec
    A = w.n_agents
    kb = synth.kv_bf16(w.seed, 501, A, w.n_kv_heads, w.d_qk)
    vb = None if w.v_aliases_k else synth.kv_bf16(w.seed, 502, A, w.n_kv_heads, w.d_v)
    q = synth.normal_bf16(w.seed, 7, (A, w.n_q_heads, w.d_qk))
    lens1 = [n + 1 for n in w.lens]
    offs = np.arange(A + 1, dtype=np.int32)
    O.quantize_append(p.opool, 0, p.tabs, w.lens, offs, f32(kb), None if vb is None else f32(vb))
    windows = sorted({w.layer_window(l) for l in range(w.n_layers)})          # window layers and global layers
    import bench
    fused = bench.fused_update_and_fetch(w)               # all three take the update-and-fetch call, as the benchmark does
    if not fused:
        p.dc.append(0, w.lens, offs, kb, vb)
    for n_call, win in enumerate(windows):
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens1, win, f32(q), w.softmax_scale)
        if fused:
            out, lse = p.dc.append_decode(0, lens1, win, kb, vb, q, w.softmax_scale)   # idempotent: same token, same slot
        else:
            out, lse = p.dc.decode(0, lens1, win, q, w.softmax_scale)
        assert_attention_close(out.cpu().numpy(), ref, f"{w.name} window {win}")
        assert_lse_close(lse.cpu().numpy(), lse_ref, w.name)
    p.lens = lens1
    p.check_packed_equal()
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("index", [4, 6])
def test_full_size_prefill_launch_matches_the_oracle_on_sampled_rows(H, index):
    """Configuration 5 (and the d = 256 phase of bench workload 6) as bench.py launches it, one layer: eight agents,
    8192 cached + 1024 new tokens each (4096 + 512 at d = 256).  The library computes every output row; the oracle
    checks 24 query rows per agent (all heads), spread over the phase and including its first and last token, for two
    of the agents, and the appended cache bytes of all."""
    w = synth.workload(index)
    p = WorkloadPair(H, w, extra_tokens=w.new_tokens).fill(chunks=[max(w.lens)])
    A, T = w.n_agents, w.new_tokens
    kb = synth.kv_bf16(w.seed, 501, A * T, w.n_kv_heads, w.d_qk)
    vb = synth.kv_bf16(w.seed, 502, A * T, w.n_kv_heads, w.d_v)
    q = synth.normal_bf16(w.seed, 7, (A * T, w.n_q_heads, w.d_qk))
    offs = (np.arange(A + 1) * T).astype(np.int32)
    O.quantize_append(p.opool, 0, p.tabs, w.lens, offs, f32(kb), f32(vb))
    p.dc.append(0, w.lens, offs, kb, vb)
    lens1 = [n + T for n in w.lens]
    out, lse = p.dc.prefill(0, lens1, offs, 0, q, w.softmax_scale)
    out = out.cpu().numpy()
    local = sorted(set([0, 1, 31, 32, 63, 64, T - 1] + list(range(17, T, 61))))[:24]
    rows = [a * T + i for a in (0, A - 1) for i in local]
    ref, lse_ref = O.prefill_attention(p.opool, 0, p.tabs, lens1, offs, 0, f32(q), w.softmax_scale, rows=rows)
    assert_attention_close(out[rows], ref[rows], w.name)
    assert_lse_close(lse.cpu().numpy()[rows], lse_ref[rows], w.name)
    assert np.all(np.isfinite(out))
    p.lens = lens1
    p.check_packed_equal()
    assert p.dc.read_flags() == 0
