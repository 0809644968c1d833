"""Pins for the oracle's block-table gather, attention and pack/unpack (CPU only).

Nothing here calls the CUDA path.  The oracle is pinned by brute force written
independently (pure Python loops over nibbles), closed forms (one-hot keys,
equal keys, single key), invariances (batching, block permutation, GQA
replication, window truncation, chunking) and a library softmax cross-check.
"""
import math

import numpy as np
import pytest
import torch

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth


def f32(bits):
    return synth.bf16_bits_to_f32(bits)


def build_cache(spec, lens, seed, n_blocks=None, gain=1.0, fill=0xDEADBEEF):
    """Quantize seeded K/V into a pool through shuffled block tables. Returns pool, tables."""
    need = sum(-(-n // 256) for n in lens)
    n_blocks = n_blocks or need + 3
    pool = O.Pool(spec, n_blocks, fill=fill)
    tabs = synth.block_tables(seed, 99, lens, n_blocks)
    for l in range(spec.n_layers):
        for a, n in enumerate(lens):
            k = f32(synth.kv_bf16(seed, 1000 * l + 10 * a + 1, n, spec.n_kv_heads, spec.d_qk)) * np.float32(gain)
            v = None
            if not spec.v_aliases_k:
                v = f32(synth.kv_bf16(seed, 1000 * l + 10 * a + 2, n, spec.n_kv_heads, spec.d_v)) * np.float32(gain)
            O.quantize_append(pool, l, tabs[a:a + 1], [0], [0, n], k, v)
    return pool, tabs


def queries(seed, stream, n, spec):
    return f32(synth.normal_bf16(seed, stream, (n, spec.n_q_heads, spec.d_qk)))


# ---- brute force, written without any oracle helper ------------------------------------------
def brute_decode(pool, layer, tabs, kv_lens, window, q, scale):
    s = pool.spec
    n_rep = s.n_q_heads // s.n_kv_heads
    out = np.zeros((len(kv_lens), s.n_q_heads, s.d_v))
    for a, n in enumerate(kv_lens):
        lo = max(0, n - window) if window > 0 else 0
        for h in range(s.n_q_heads):
            hk = h // n_rep
            logits, vals = [], []
            for j in range(lo, n):
                b, slot = int(tabs[a][j // 256]), j % 256
                dot = 0.0
                krow = []
                for d in range(s.d_qk):
                    word = int(pool.Kc[layer, b, hk, slot, d // 8])
                    code = (word >> (4 * (d % 8))) & 15
                    kd = code * float(pool.Ks[layer, b, hk, slot, d // 64]) + float(pool.Kb[layer, b, hk, slot, d // 64])
                    krow.append(kd)
                    dot += float(q[a, h, d]) * kd
                logits.append(scale * dot)
                if s.v_aliases_k:
                    vals.append(krow[: s.d_v])
                else:
                    vrow = []
                    for d in range(s.d_v):
                        word = int(pool.Vc[layer, b, hk, slot, d // 8])
                        code = (word >> (4 * (d % 8))) & 15
                        vrow.append(code * float(pool.Vs[layer, b, hk, slot, d // 64]) + float(pool.Vb[layer, b, hk, slot, d // 64]))
                    vals.append(vrow)
            m = max(logits)
            w = [math.exp(x - m) for x in logits]
            z = sum(w)
            for d in range(s.d_v):
                out[a, h, d] = sum(w[i] * vals[i][d] for i in range(len(w))) / z
    return out


@pytest.mark.parametrize("alias", [False, True])
def test_decode_matches_brute_force_tiny(alias):
    spec = O.Spec(2, 4, 2, 64, 64, v_aliases_k=alias)
    lens = [300, 17]                                   # spans two blocks and a ragged tail
    pool, tabs = build_cache(spec, lens, seed=5)
    q = queries(5, 7, 2, spec)
    kv = [min(n, 20) if a else n for a, n in enumerate(lens)]
    # keep brute force small: agent 0 with a 12-token window crossing the block boundary region
    out_o, _ = O.decode_attention(pool, 1, tabs, [262, 17], 12, q, 0.3)
    out_b = brute_decode(pool, 1, tabs, [262, 17], 12, q, 0.3)
    assert np.max(np.abs(out_o - out_b)) < 1e-12
    out_o, _ = O.decode_attention(pool, 0, tabs, [20, 9], 0, q, 0.125)
    out_b = brute_decode(pool, 0, tabs, [20, 9], 0, q, 0.125)
    assert np.max(np.abs(out_o - out_b)) < 1e-12


# ---- closed forms ------------------------------------------------------------------------------
def test_one_hot_keys_select_one_value_row():
    spec = O.Spec(1, 2, 1, 64, 64)
    n = 40
    perm = synth.rng(3, 0).permutation(64)[:n]
    k = np.zeros((n, 1, 64), dtype=np.float32)
    k[np.arange(n), 0, perm] = 7.5                      # 15 * 0.5: quantizes exactly (scale 0.5, bias 0)
    v = f32(synth.kv_bf16(3, 1, n, 1, 64))
    pool = O.Pool(spec, 2)
    tabs = np.array([[1, -1]], dtype=np.int32)
    O.quantize_append(pool, 0, tabs, [0], [0, n], k, v)
    Kd, Vd = O.gather_dequant(pool, 0, tabs[0], 0, n, 0)
    assert np.array_equal(Kd, k[:, 0].astype(np.float64))
    for m in (0, 13, 39):
        q = np.zeros((1, 2, 64), dtype=np.float32)
        q[0, :, perm[m]] = 16.0                         # logit gap 16*7.5*1 = 120 -> exp(-120) leakage
        out, lse = O.decode_attention(pool, 0, tabs, [n], 0, q, 1.0)
        assert np.max(np.abs(out[0, 0] - Vd[m])) < 1e-40 + 40 * math.exp(-120) * 10
        assert abs(lse[0, 0] - 120.0) < 1e-9


def test_equal_keys_or_zero_scale_give_mean_of_values_and_single_key_gives_that_row():
    spec = O.Spec(1, 4, 2, 128, 128)
    n = 77
    k = np.tile(f32(synth.kv_bf16(4, 1, 1, 2, 128)), (n, 1, 1))
    v = f32(synth.kv_bf16(4, 2, n, 2, 128))
    pool = O.Pool(spec, 1)
    tabs = np.array([[0]], dtype=np.int32)
    O.quantize_append(pool, 0, tabs, [0], [0, n], k, v)
    q = queries(4, 3, 1, spec)
    out, lse = O.decode_attention(pool, 0, tabs, [n], 0, q, 0.2)
    for h in range(4):
        _, Vd = O.gather_dequant(pool, 0, tabs[0], 0, n, h // 2)
        assert np.max(np.abs(out[0, h] - Vd.mean(axis=0))) < 1e-13
    # softmax_scale = 0 on arbitrary keys: uniform weights, lse = ln n
    pool2, tabs2 = build_cache(spec, [n], seed=6)
    out2, lse2 = O.decode_attention(pool2, 0, tabs2, [n], 0, q, 0.0)
    _, Vd = O.gather_dequant(pool2, 0, tabs2[0], 0, n, 1)
    assert np.max(np.abs(out2[0, 3] - Vd.mean(axis=0))) < 1e-13
    assert abs(lse2[0, 3] - math.log(n)) < 1e-12
    # kv_len = 1: the output is V row 0 exactly
    out1, _ = O.decode_attention(pool2, 0, tabs2, [1], 0, q, 0.7)
    assert np.array_equal(out1[0, 3], Vd[0])
    # kv_len = 0: zeros and lse = -inf
    out0, lse0 = O.decode_attention(pool2, 0, tabs2, [0], 0, q, 0.7)
    assert np.all(out0 == 0) and np.all(np.isneginf(lse0))


def test_softmax_weights_sum_to_one_and_match_library_softmax():
    spec = O.Spec(1, 8, 2, 128, 128)
    lens = [1000, 700]
    pool, tabs = build_cache(spec, lens, seed=8)
    q = queries(8, 5, 2, spec)
    scale = 1 / math.sqrt(128)
    out, lse = O.decode_attention(pool, 0, tabs, lens, 0, q, scale)
    for a in range(2):
        for h in (0, 5):
            K, V = O.gather_dequant(pool, 0, tabs[a], 0, lens[a], h // 4)
            logits = scale * (K @ q[a, h].astype(np.float64))
            assert abs(np.exp(logits - lse[a, h]).sum() - 1.0) < 1e-12
            ref = torch.softmax(torch.from_numpy(logits), dim=0) @ torch.from_numpy(V)
            assert np.max(np.abs(out[a, h] - ref.numpy())) < 1e-12


# ---- invariances -------------------------------------------------------------------------------
def test_batched_equals_per_agent_and_block_permutation_is_invisible():
    spec = O.Spec(1, 4, 2, 64, 64)
    lens = [515, 100, 256]
    pool, tabs = build_cache(spec, lens, seed=9)
    q = queries(9, 5, 3, spec)
    out, lse = O.decode_attention(pool, 0, tabs, lens, 0, q, 0.1)
    for a in range(3):
        o1, l1 = O.decode_attention(pool, 0, tabs[a:a + 1], lens[a:a + 1], 0, q[a:a + 1], 0.1)
        assert np.array_equal(o1[0], out[a]) and np.array_equal(l1[0], lse[a])
    # same logical content behind different physical blocks
    buf = [O.pack(pool, tabs[a], lens[a]) for a in range(3)]
    pool2 = O.Pool(spec, pool.n_blocks + 4, fill=0x12345678)
    tabs2 = synth.block_tables(1234, 1, lens, pool2.n_blocks)
    assert not np.array_equal(tabs, tabs2)
    for a in range(3):
        O.unpack(pool2, tabs2[a], lens[a], buf[a])
    out2, _ = O.decode_attention(pool2, 0, tabs2, lens, 0, q, 0.1)
    assert np.array_equal(out, out2)
    for a in range(3):
        assert np.array_equal(O.pack(pool2, tabs2[a], lens[a]), buf[a])


def test_window_equals_truncated_cache_and_differs_from_global():
    spec = O.Spec(1, 2, 1, 64, 64)
    n, W = 700, 300                                    # window start 400 is not block aligned
    k = f32(synth.kv_bf16(10, 1, n, 1, 64))
    v = f32(synth.kv_bf16(10, 2, n, 1, 64))
    pool = O.Pool(spec, 4)
    tabs = np.array([[2, 0, 3]], dtype=np.int32)
    O.quantize_append(pool, 0, tabs, [0], [0, n], k, v)
    q = queries(10, 3, 1, spec)
    out_w, _ = O.decode_attention(pool, 0, tabs, [n], W, q, 0.2)
    out_g, _ = O.decode_attention(pool, 0, tabs, [n], 0, q, 0.2)
    assert np.max(np.abs(out_w - out_g)) > 1e-3
    pool_t = O.Pool(spec, 2)
    tabs_t = np.array([[1, 0]], dtype=np.int32)
    O.quantize_append(pool_t, 0, tabs_t, [0], [0, W], k[n - W:], v[n - W:])
    out_t, _ = O.decode_attention(pool_t, 0, tabs_t, [W], 0, q, 0.2)
    assert np.max(np.abs(out_w - out_t)) < 1e-14
    # a window at least as long as the cache is the global result
    out_big, _ = O.decode_attention(pool, 0, tabs, [n], n, q, 0.2)
    assert np.array_equal(out_big, out_g)


def test_gqa_equals_mha_on_replicated_kv_heads():
    spec = O.Spec(1, 6, 2, 64, 64)
    n = 90
    k = f32(synth.kv_bf16(11, 1, n, 2, 64))
    v = f32(synth.kv_bf16(11, 2, n, 2, 64))
    pool = O.Pool(spec, 1)
    tabs = np.array([[0]], dtype=np.int32)
    O.quantize_append(pool, 0, tabs, [0], [0, n], k, v)
    q = queries(11, 3, 1, spec)
    out, _ = O.decode_attention(pool, 0, tabs, [n], 0, q, 0.15)
    spec_m = O.Spec(1, 6, 6, 64, 64)
    pool_m = O.Pool(spec_m, 1)
    O.quantize_append(pool_m, 0, tabs, [0], [0, n], np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1))
    out_m, _ = O.decode_attention(pool_m, 0, tabs, [n], 0, q, 0.15)
    assert np.array_equal(out, out_m)


def test_latent_alias_equals_explicit_value_cache():
    spec_a = O.Spec(1, 4, 1, 192, 128, v_aliases_k=True)
    spec_e = O.Spec(1, 4, 1, 192, 128)
    n = 130
    k = f32(synth.kv_bf16(12, 1, n, 1, 192))
    pool_a, pool_e = O.Pool(spec_a, 1), O.Pool(spec_e, 1)
    tabs = np.array([[0]], dtype=np.int32)
    O.quantize_append(pool_a, 0, tabs, [0], [0, n], k, None)
    O.quantize_append(pool_e, 0, tabs, [0], [0, n], k, k[:, :, :128].copy())
    q = queries(12, 3, 1, spec_a)
    oa, la = O.decode_attention(pool_a, 0, tabs, [n], 0, q, 0.1)
    oe, le = O.decode_attention(pool_e, 0, tabs, [n], 0, q, 0.1)
    assert np.array_equal(oa, oe) and np.array_equal(la, le)
    assert spec_a.block_bytes() == 256 * (96 + 12)


def test_prefill_rows_equal_decode_calls_and_chunking_is_invisible():
    spec = O.Spec(1, 4, 2, 64, 64)
    P, C = 300, 40
    lens = [P + C, 70 + C]
    pool, tabs = build_cache(spec, lens, seed=13)
    q_offs = [0, C, 2 * C]
    q = queries(13, 5, 2 * C, spec)
    for W in (0, 50):
        out, lse = O.prefill_attention(pool, 0, tabs, lens, q_offs, W, q, 0.2)
        for a in range(2):
            for i in (0, 1, C // 2, C - 1):
                row = q_offs[a] + i
                od, ld = O.decode_attention(pool, 0, tabs[a:a + 1], [lens[a] - C + i + 1], W, q[row][None], 0.2)
                assert np.max(np.abs(od[0] - out[row])) < 1e-14
                assert np.max(np.abs(ld[0] - lse[row])) < 1e-12
        # two chunks of C/2 (second call sees the full cache, first call a cache shorter by C/2)
        h = C // 2
        q1 = np.concatenate([q[0:h], q[C:C + h]])
        q2 = np.concatenate([q[h:C], q[C + h:2 * C]])
        o1, _ = O.prefill_attention(pool, 0, tabs, [n - h for n in lens], [0, h, 2 * h], W, q1, 0.2)
        o2, _ = O.prefill_attention(pool, 0, tabs, lens, [0, h, 2 * h], W, q2, 0.2)
        assert np.array_equal(np.concatenate([o1[:h], o2[:h], o1[h:], o2[h:]]), out)
    # causal: the first new query must not see later new tokens
    out_full, _ = O.prefill_attention(pool, 0, tabs, lens, q_offs, 0, q, 0.2)
    od, _ = O.decode_attention(pool, 0, tabs[:1], [lens[0]], 0, q[0][None], 0.2)
    assert np.max(np.abs(od[0] - out_full[0])) > 1e-4
    # rows= computes only the sampled rows
    sub, _ = O.prefill_attention(pool, 0, tabs, lens, q_offs, 0, q, 0.2, rows=[3, C + 7])
    assert np.array_equal(sub[3], out_full[3]) and np.array_equal(sub[C + 7], out_full[C + 7])
    assert np.all(sub[4] == 0)


def test_append_then_attend_sees_the_new_token_in_quantized_form():
    spec = O.Spec(1, 2, 1, 64, 64)
    n = 255                                             # the appended token opens nothing new; 256 would
    pool, tabs = build_cache(spec, [n + 2], seed=14)
    pool.Kc[0, tabs[0, 0], :, n:] = 0xFFFFFFFF          # stale garbage beyond the length
    knew = f32(synth.kv_bf16(14, 50, 2, 1, 64))
    vnew = f32(synth.kv_bf16(14, 51, 2, 1, 64))
    O.quantize_append(pool, 0, tabs, [n], [0, 2], knew, vnew)   # crosses into the second block
    K, V = O.gather_dequant(pool, 0, tabs[0], n, n + 2, 0)
    c, s, b = O.quantize_rows(vnew[:, 0])
    assert np.array_equal(V, O.dequantize(c, s, b))
    assert np.max(np.abs(V - vnew[:, 0])) <= float(s.max()) / 2 * 1.00001
    q = queries(14, 3, 1, spec)
    o_before, _ = O.decode_attention(pool, 0, tabs, [n], 0, q, 0.2)
    o_after, _ = O.decode_attention(pool, 0, tabs, [n + 2], 0, q, 0.2)
    assert np.max(np.abs(o_before - o_after)) > 1e-6


def test_unpack_rejects_wrong_size_and_pack_roundtrip_is_identity():
    spec = O.Spec(3, 2, 2, 64, 128)                     # asymmetric d_k != d_v
    lens = [600]
    pool, tabs = build_cache(spec, lens, seed=15)
    buf = O.pack(pool, tabs[0], 600)
    assert buf.size == 3 * 3 * 256 * 2 * (32 + 4 + 64 + 8)
    pool2 = O.Pool(spec, 7, fill=0xABABABAB)
    row = np.array([6, 2, 4], dtype=np.int32)
    O.unpack(pool2, row, 600, buf)
    assert np.array_equal(O.pack(pool2, row, 600), buf)
    with pytest.raises(AssertionError):
        O.unpack(pool2, row, 600, buf[:-1])
