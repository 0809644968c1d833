"""GPU parity for caches whose scales and biases are bfloat16 (Section 3.2 and Appendix "safetensors Q4 Format": the
type the paper persisted for two of its three models).  Same bars as the binary16 tests: cache bytes bit-exact,
attention within 2e-3 absolute and 1e-2 row-relative of the float64 oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth
from test_gpu_parity import (H, SPECS, Pair, TiePair, assert_attention_close, assert_lse_close, f32)  # noqa: F401

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", list(SPECS))
def test_quantize_append_and_pack_bit_exact(H, name):
    p = Pair(H, SPECS[name], [300, 17, 256], seed=121, sb_dtype=1)
    p.fill(chunks=[5, 1, 2, 40, 1, 300])          # single-token launches, partial octets and the bulk kernel
    p.check_packed_equal()


def test_adversarial_values_and_rounding_boundaries_bit_exact(H):
    p = Pair(H, SPECS["gqa128"], [64], seed=122, sb_dtype=1)
    s = p.ospec
    x = synth.rng(122, 5).standard_normal((64, s.n_kv_heads, s.d_qk), dtype=np.float32)
    x[1] *= 100.0
    x[2] = 1000.0 + 0.01 * x[2]
    x[3, :, :64] = 3.0
    x[4] *= 1e-6
    x[5, 0, 5] = 65280.0
    x[5, 0, 6] = -65280.0
    x[6] = 0.0
    x[7, :, 0] = -0.0
    x[8] *= 1e-30                                  # far below binary16's range: bfloat16 keeps it
    x[9] = np.round(x[9] * 2) / 2
    kb = synth.f32_to_bf16_bits(x)
    vb = synth.f32_to_bf16_bits(x[::-1].copy())
    for l in range(s.n_layers):
        O.quantize_append(p.opool, l, p.tabs, [0], [0, 64], f32(kb), f32(vb))
        p.dc.append(l, [0], [0, 64], kb, vb)
    p.check_packed_equal()
    assert np.any(p.opool.Ks[0, p.tabs[0][0], :, 8] != 0)      # the tiny row did not collapse to scale 0
    t = TiePair(H, SPECS["gqa128"], [300, 70], seed=123, sb_dtype=1).fill(chunks=[3, 64, 300])
    t.check_packed_equal()


@pytest.mark.parametrize("name,lens,window", [
    ("gqa64", [300, 17, 262], 12),
    ("gqa128", [1000, 700, 1, 255, 256, 257], 0),
    ("gqa128", [1000, 700, 33], 300),
    ("gqa256", [1500, 1100], 1024),
    ("mla", [600, 70], 0),
    ("asym", [400, 300], 100),
])
def test_decode_matches_oracle(H, name, lens, window):
    p = Pair(H, SPECS[name], lens, seed=131, sb_dtype=1).fill()
    s = p.ospec
    q = p.q(7, len(lens))
    scale = 1.0 / math.sqrt(s.d_qk if name != "mla" else 192)
    for l in range(s.n_layers):
        ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, lens, window, f32(q), scale)
        out, lse = p.dc.decode(l, lens, window, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"{name} layer {l}")
        assert_lse_close(lse.cpu().numpy(), lse_ref, name)
    assert p.dc.read_flags() == 0


def test_decode_long_context_wraps_the_ring(H):
    spec_args, lens = (1, 32, 8, 128, 128, False), [40000, 23000]
    p = Pair(H, spec_args, lens, seed=137, sb_dtype=1).fill()
    q = p.q(7, len(lens))
    ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), 1.0 / math.sqrt(128))
    out, lse = p.dc.decode(0, lens, 0, q, 1.0 / math.sqrt(128))
    assert_attention_close(out.cpu().numpy(), ref)
    assert_lse_close(lse.cpu().numpy(), lse_ref)
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("name,lens,window", [
    ("gqa128", [1000, 700, 0, 255, 256, 257, 31, 32, 33], 0),
    ("gqa256", [1500, 41, 2049], 1024),
    ("asym", [700, 33, 0, 256], 0),
])
def test_update_and_fetch_in_one_launch(H, name, lens, window):
    steps = 3
    p = Pair(H, SPECS[name], lens, seed=139, extra_tokens=steps, sb_dtype=1).fill()
    s = p.ospec
    A = len(lens)
    cur = list(lens)
    scale = 1.0 / math.sqrt(s.d_qk)
    for step in range(steps):
        kb = synth.kv_bf16(139, 500 + step, A, s.n_kv_heads, s.d_qk)
        vb = synth.kv_bf16(139, 600 + step, A, s.n_kv_heads, s.d_v)
        q = p.q(70 + step, A)
        live = [a for a in range(A) if lens[a] > 0]
        new_lens = [n + 1 if lens[a] > 0 else 0 for a, n in enumerate(cur)]
        for l in range(s.n_layers):
            offs = np.concatenate([[0], np.cumsum([1 if a in live else 0 for a in range(A)])]).astype(np.int32)
            O.quantize_append(p.opool, l, p.tabs, cur, offs, f32(kb[live]), f32(vb[live]))
            ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, new_lens, window, f32(q), scale)
            out, lse = p.dc.append_decode(l, new_lens, window, kb, vb, q, scale)
            assert_attention_close(out.cpu().numpy(), ref, f"{name} step {step} layer {l}")
            assert_lse_close(lse.cpu().numpy(), lse_ref, name)
        cur = new_lens
    p.lens = cur
    p.check_packed_equal()
    assert p.dc.read_flags() == 0


def test_latent_cache_update_and_fetch(H):
    """A bfloat16 latent cache through both entries: the step's new row quantized with bfloat16 scale and bias by the
    attention kernel itself, pool bytes as quantize-append writes them."""
    lens = [300, 64, 1000]
    steps = 2
    p = Pair(H, SPECS["mla"], lens, seed=140, extra_tokens=steps, sb_dtype=1).fill()
    s = p.ospec
    A = len(lens)
    cur = list(lens)
    scale = 1.0 / math.sqrt(192)
    for step in range(steps):
        kb = synth.kv_bf16(140, 500 + step, A, s.n_kv_heads, s.d_qk)
        q = p.q(70 + step, A)
        new_lens = [n + 1 for n in cur]
        O.quantize_append(p.opool, 0, p.tabs, cur, list(range(A + 1)), f32(kb), None)
        ref, lse_ref = O.decode_attention(p.opool, 0, p.tabs, new_lens, 0, f32(q), scale)
        out, lse = p.dc.append_decode(0, new_lens, 0, kb, None, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"step {step}")
        assert_lse_close(lse.cpu().numpy(), lse_ref)
        out, lse = p.dc.decode(0, new_lens, 0, q, scale)
        assert_attention_close(out.cpu().numpy(), ref, f"two calls, step {step}")
        cur = new_lens
    for l in range(1, s.n_layers):                              # the other layers get the same rows through quantize-append
        for step in range(steps):
            kb = synth.kv_bf16(140, 500 + step, A, s.n_kv_heads, s.d_qk)
            O.quantize_append(p.opool, l, p.tabs, [n + step for n in lens], list(range(A + 1)), f32(kb), None)
            p.dc.append(l, [n + step for n in lens], list(range(A + 1)), kb, None)
    p.lens = cur
    p.check_packed_equal()
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("name,prefix,chunk,window", [
    ("gqa64", [300, 70], 40, 50),
    ("gqa128", [512, 200], 130, 0),
    ("gqa128", [300, 0], 70, 100),
    ("gqa256", [256, 10], 70, 128),
    ("gqa256", [900, 0], 150, 0),
    ("asym", [900, 0, 63], 150, 0),
    ("asym", [300, 70], 40, 50),
])
def test_prefill_matches_oracle(H, name, prefix, chunk, window):
    lens = [n + chunk for n in prefix]
    p = Pair(H, SPECS[name], lens, seed=141, sb_dtype=1).fill(chunks=[max(prefix), chunk])
    s = p.ospec
    A = len(lens)
    q_offs = [chunk * a for a in range(A + 1)]
    q = p.q(7, chunk * A)
    scale = 1.0 / math.sqrt(s.d_qk)
    ref, lse_ref = O.prefill_attention(p.opool, 0, p.tabs, lens, q_offs, window, f32(q), scale)
    out, lse = p.dc.prefill(0, lens, q_offs, window, q, scale)
    assert_attention_close(out.cpu().numpy(), ref, name)
    assert_lse_close(lse.cpu().numpy(), lse_ref, name)
    assert p.dc.read_flags() == 0


def test_values_outside_the_binary16_range_of_scales(H):
    """Rows of magnitude 1e-9 give scales near 1e-10, below binary16's smallest subnormal: bfloat16 keeps them.  The
    shape-agnostic kernel (float32 throughout) follows them to relative accuracy; the tensor-core kernel carries
    probability x scale as binary16 pairs, so there its stated bound is the absolute one (2e-5 M + 1e-5)."""
    lens = [200, 40]
    for name in ("gqa64", "gqa128"):
        p = Pair(H, SPECS[name], lens, seed=142, gain=1e-9, sb_dtype=1).fill()
        sv = O.sb_values(p.opool.Vs[0, p.tabs[0][0], :, :200])
        assert np.all(sv > 0) and sv.max() < 6e-8
        q = p.q(7, 2)
        scale = 1.0 / math.sqrt(p.ospec.d_qk)
        ref, _ = O.decode_attention(p.opool, 0, p.tabs, lens, 0, f32(q), scale)
        out, _ = p.dc.decode(0, lens, 0, q, scale)
        got = out.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(ref)) > 1e-11
        if name == "gqa64":
            assert np.max(np.abs(got - ref)) <= 1e-3 * np.max(np.abs(ref))
        else:
            assert np.max(np.abs(got - ref)) <= 1e-5
        assert p.dc.read_flags() == 0


@pytest.mark.parametrize("name,lens", [("gqa128", [700, 33]), ("mla", [300, 256])])
def test_saved_image_names_bf16_and_restores(H, name, lens):
    p = Pair(H, SPECS[name], lens, seed=161, sb_dtype=1).fill()
    p2 = Pair(H, SPECS[name], lens, seed=162, sb_dtype=1)
    for a, n in enumerate(lens):
        img = p.dc.save(a, n)
        ref = O.container(p.opool, p.tabs[a], n)
        assert img.numel() == ref.size and np.array_equal(img.numpy(), ref), f"agent {a}"
        assert b'"dtype":"BF16"' in img.numpy().tobytes()[:4096]
        assert p2.dc.restore(a, img.pin_memory(), staging_layers=1) == n
        assert np.array_equal(p2.dc.pack(a, n).cpu().numpy(), O.pack(p.opool, p.tabs[a], n))
    # an image of one type is not restored into a cache of the other
    from paper_2603_04428_b200 import binding as B
    p3 = Pair(H, SPECS[name], lens, seed=163, sb_dtype=0)
    with pytest.raises(B.Q4KVError):
        p3.dc.restore(0, p.dc.save(0, lens[0]).pin_memory(), staging_layers=1)
    assert p.dc.read_flags() == 0 and p2.dc.read_flags() == 0


def test_layer_batched_entry_and_static_entry(H):
    """The layer-batched entry and the entry without a caller workspace on a bfloat16 cache."""
    from paper_2603_04428_b200 import binding as B
    spec_args, lens = (3, 8, 2, 128, 128, False), [700, 33, 300]
    p = Pair(H, spec_args, lens, seed=171, sb_dtype=1).fill()
    s = p.ospec
    L, A = s.n_layers, len(lens)
    scale = 1.0 / math.sqrt(s.d_qk)
    q_all = np.stack([p.q(80 + l, A) for l in range(L)])
    out = torch.full((L, A, s.n_q_heads, s.d_v), float("nan"), device="cuda")
    lse = torch.full((L, A, s.n_q_heads), float("nan"), device="cuda")
    ws = torch.zeros(B.q4kv_workspace_bytes_layers(p.dc.spec, A, p.dc.bt.max_blocks * 256, L), dtype=torch.uint8, device="cuda")
    lens_d = H.dev(np.asarray(lens, dtype=np.int32))
    B.q4kv_decode_attention_layers(p.dc.spec, p.dc.pool, p.dc.n_blocks, 0, L, p.dc.bt, lens_d, 0, [0] * L, None, None,
                                   H.bf16_dev(q_all), scale, out, B.OUT_F32, lse, ws, p.dc.flags)
    out_s = torch.full((A, s.n_q_heads, s.d_v), float("nan"), device="cuda")
    for l in range(L):
        ref, lse_ref = O.decode_attention(p.opool, l, p.tabs, lens, 0, f32(q_all[l]), scale)
        assert_attention_close(out[l].cpu().numpy(), ref, f"layer {l}")
        assert_lse_close(lse[l].cpu().numpy(), lse_ref)
        B.q4kv_decode_attention_static(p.dc.spec, p.dc.pool, p.dc.n_blocks, l, p.dc.bt, lens_d, 0, 0, H.bf16_dev(q_all[l]),
                                       scale, out_s, B.OUT_F32, None, p.dc.flags)
        assert_attention_close(out_s.cpu().numpy(), ref, f"static entry, layer {l}")
    assert p.dc.read_flags() == 0


@pytest.mark.parametrize("name", ["gqa128", "gqa256", "asym", "mla"])
def test_a_scale_beyond_binary16_is_reported_by_the_tile_kernels(H, name):
    """The library's own quantizer never produces a scale or bias beyond binary16's largest number (its inputs are
    bounded by it, and the header asks the same of caches persisted elsewhere), but nothing stops a foreign file from
    holding one.  Such a scale (here 2^20, planted in the oracle's pool and carried to the device through pack /
    unpack) cannot enter a binary16 tile: the kernels that build such tiles raise Q4KV_FLAG_SB_RANGE rather than
    return a wrong result silently; the same planted value past the agent's length is not looked at."""
    from paper_2603_04428_b200 import binding as B
    lens = [300, 64]
    chunk = 40
    p = Pair(H, SPECS[name], [n + chunk for n in lens], seed=150, sb_dtype=1).fill()
    s = p.ospec
    latent = bool(s.v_aliases_k)
    q_offs = [chunk * a for a in range(len(lens) + 1)]
    q = p.q(7, len(lens) if latent else chunk * len(lens))
    scale = 1.0 / math.sqrt(192 if latent else s.d_qk)

    def attend():
        if latent:
            return p.dc.decode(0, p.lens, 0, q, scale)[0]
        return p.dc.prefill(0, p.lens, q_offs, 0, q, scale)[0]

    good = attend()
    assert p.dc.read_flags() == 0
    blk = int(p.tabs[0][1])                            # agent 0's second block holds tokens 256 .. 339
    for tok, expect in ((340 - 256 + 3, False), (17, True)):     # past the length: ignored; inside: reported
        (p.opool.Ks if latent else p.opool.Vs)[0, blk, 0, tok, 0] = 0x4980     # 2^20 as bfloat16
        p.dc.unpack(0, 512, O.pack(p.opool, p.tabs[0], 512))
        out = attend()
        flags = p.dc.read_flags()
        assert bool(flags & B.FLAG_SB_RANGE) == expect and (flags & ~B.FLAG_SB_RANGE) == 0
        if not expect:
            assert torch.equal(out, good)
        p.dc.flags.zero_()
