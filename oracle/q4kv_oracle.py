"""CPU oracle for the Q4 KV-cache hot path.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain definition the CUDA library is checked against.
It is imported only by the tests, by the smoke check and by the benchmark's CPU
baseline leg; the product never routes through it and shares no code with it.

What it follows (paper sections, not code):
  * Q4 element format -- Section 3.2 "Q4 Quantization Pipeline": 4-bit codes,
    eight per uint32, plus a 16-bit scale and bias per group of g = 64
    consecutive head-dim elements; K+V bytes per layer = h*d*n*(1 + 8/g).
  * Block pool -- Section 3.1: fixed 256-token blocks, one list of blocks per
    agent and layer (here: a per-agent block table of physical block ids).
  * update-then-attend over the whole quantized cache, batched over agents --
    Section 3.4 "Batched Quantized Inference"; GQA head mapping and
    sliding-window layers -- Section 3.6 "Architectural Coverage".
  * Chunked prefill / cross-phase injection -- Sections 3.4 and 3.5: new
    queries attend the cached prefix plus the causal new tokens.
  * Persisted per-block tensor schema -- Appendix A.

The paper delegates the quantizer's exact arithmetic to a library, so the
sequence below is this library's fixed reading (single binary32 operations in the
order written; bias rounded down, scale rounded up to binary16 so that the code
range always covers the group's range).  Attention is the textbook definition
in float64 over the dequantized values.

Parity status: every function here is pinned by tests/test_oracle_*.py
(closed forms, hand-worked literals, brute force, invariants).  The effect of
Q4 on model perplexity (Table 8) is "parity unpinned": it needs weights and a
corpus and is not a target.
"""
from __future__ import annotations

import numpy as np

GROUP = 64          # elements per quantization group (Section 3.2)
BLOCK_TOKENS = 256  # tokens per pool block (Section 3.1)


# ----------------------------------------------------------------------------
# number formats
# ----------------------------------------------------------------------------
def _f16_round_down(x32: np.ndarray) -> np.ndarray:
    """binary32 -> binary16, rounding toward -infinity."""
    h = x32.astype(np.float16)                       # round to nearest first
    too_big = h.astype(np.float32) > x32
    h = np.where(too_big, np.nextafter(h, np.float16(-np.inf)), h)
    return h.astype(np.float16)


def _f16_round_up(x32: np.ndarray) -> np.ndarray:
    """binary32 -> binary16, rounding toward +infinity."""
    h = x32.astype(np.float16)
    too_small = h.astype(np.float32) < x32
    h = np.where(too_small, np.nextafter(h, np.float16(np.inf)), h)
    return h.astype(np.float16)


def _bf16_round_down(x32: np.ndarray) -> np.ndarray:
    """binary32 -> bfloat16 bit patterns (uint16), rounding toward -infinity.

    bfloat16 is the upper half of binary32, so dropping the lower 16 bits rounds toward zero; a negative value that
    lost bits moves one step further from zero."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    top = u >> np.uint32(16)
    lost = (u & np.uint32(0xFFFF)) != 0
    neg = (u >> np.uint32(31)) != 0
    return (top + (lost & neg)).astype(np.uint16)


def _bf16_round_up(x32: np.ndarray) -> np.ndarray:
    """binary32 -> bfloat16 bit patterns (uint16), rounding toward +infinity."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    top = u >> np.uint32(16)
    lost = (u & np.uint32(0xFFFF)) != 0
    neg = (u >> np.uint32(31)) != 0
    return (top + (lost & ~neg)).astype(np.uint16)


def sb_values(a: np.ndarray) -> np.ndarray:
    """Scales or biases as float64 numbers: float16 arrays hold binary16 values, uint16 arrays bfloat16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    assert a.dtype == np.float16
    return a.astype(np.float64)


# ----------------------------------------------------------------------------
# quantizer (Section 3.2 format; arithmetic = this library's fixed reading)
# ----------------------------------------------------------------------------
def quantize_rows(x32: np.ndarray, sb_dtype: int = 0):
    """Quantize rows of binary32 values (already exact images of bf16 inputs).

    x32: [..., D] float32, D a multiple of 64, finite, |x| <= 65504.
    Returns (codes uint8 [..., D] in 0..15, scale [..., D/64], bias [..., D/64]);
    scale and bias are float16 arrays for sb_dtype 0 (binary16) and uint16 arrays of
    bfloat16 bit patterns for sb_dtype 1 (Section 3.2 and Appendix A name both types);
    the sequence is the same with the 16-bit roundings taken in that type.
    Per group of 64 consecutive elements:
        bias  = round_down_f16(min x)            (a zero result is stored as +0)
        r     = f32(max x - f32(bias))
        scale = round_up_f16(f32(r / 15))
        code  = clamp(round_half_even(f32(f32(x - f32(bias)) / f32(scale))), 0, 15)
        (scale == 0  ->  all codes 0)
    """
    x32 = np.asarray(x32, dtype=np.float32)
    D = x32.shape[-1]
    assert D % GROUP == 0
    assert np.all(np.isfinite(x32)) and np.all(np.abs(x32) <= np.float32(65504.0))
    xg = x32.reshape(x32.shape[:-1] + (D // GROUP, GROUP))
    mn = xg.min(axis=-1)
    mx = xg.max(axis=-1)
    if sb_dtype == 0:
        bias = _f16_round_down(mn)
        bias = np.where(bias == np.float16(0), np.float16(0), bias).astype(np.float16)
    else:
        assert sb_dtype == 1
        bias = _bf16_round_down(mn)
        bias = np.where(bias == np.uint16(0x8000), np.uint16(0), bias).astype(np.uint16)
    bias32 = sb_values(bias).astype(np.float32)          # exact: both 16-bit types embed in binary32
    r = (mx - bias32).astype(np.float32)
    r15 = (r / np.float32(15.0)).astype(np.float32)
    scale = _f16_round_up(r15) if sb_dtype == 0 else _bf16_round_up(r15)
    scale32 = sb_values(scale).astype(np.float32)
    safe = np.where(scale32 == 0, np.float32(1.0), scale32)
    t = ((xg - bias32[..., None]).astype(np.float32) / safe[..., None]).astype(np.float32)
    c = np.clip(np.rint(t), 0, 15)
    c = np.where(scale32[..., None] == 0, 0, c).astype(np.uint8)
    return c.reshape(x32.shape), scale, bias


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """[..., D] codes -> [..., D/8] uint32; element k of each eight sits in bits [4k, 4k+4)."""
    c = np.asarray(codes, dtype=np.uint32)
    c8 = c.reshape(c.shape[:-1] + (c.shape[-1] // 8, 8))
    w = np.zeros(c8.shape[:-1], dtype=np.uint32)
    for k in range(8):
        w |= c8[..., k] << np.uint32(4 * k)
    return w


def unpack_codes(words: np.ndarray) -> np.ndarray:
    """Inverse of pack_codes: [..., W] uint32 -> [..., 8W] uint8."""
    w = np.asarray(words, dtype=np.uint32)
    out = np.empty(w.shape + (8,), dtype=np.uint8)
    for k in range(8):
        out[..., k] = (w >> np.uint32(4 * k)) & np.uint32(15)
    return out.reshape(w.shape[:-1] + (w.shape[-1] * 8,))


def dequantize(codes: np.ndarray, scale: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """x_hat = code * scale + bias in float64 (4-bit x 11-bit + 11-bit; exact, or at most one rounding of the sum)."""
    D = codes.shape[-1]
    cg = codes.reshape(codes.shape[:-1] + (D // GROUP, GROUP)).astype(np.float64)
    xh = cg * sb_values(scale)[..., None] + sb_values(bias)[..., None]
    return xh.reshape(codes.shape)


# ----------------------------------------------------------------------------
# cache spec, pool, block tables (Sections 3.1, 3.6; Appendix A)
# ----------------------------------------------------------------------------
class Spec:
    """Architectural parameters of one model's cache (the paper's ModelCacheSpec)."""

    def __init__(self, n_layers, n_q_heads, n_kv_heads, d_qk, d_v, v_aliases_k=False, sb_dtype=0):
        assert n_q_heads % n_kv_heads == 0 and d_qk % GROUP == 0 and d_v % GROUP == 0
        assert sb_dtype in (0, 1)                        # scale / bias type: 0 binary16, 1 bfloat16
        if v_aliases_k:
            assert d_v <= d_qk
        self.n_layers, self.n_q_heads, self.n_kv_heads = n_layers, n_q_heads, n_kv_heads
        self.d_qk, self.d_v, self.v_aliases_k = d_qk, d_v, bool(v_aliases_k)
        self.sb_dtype = sb_dtype

    @property
    def n_rep(self):
        return self.n_q_heads // self.n_kv_heads

    def row_bytes(self):
        """Bytes of one token's K and V over all KV heads (codes + scales + biases)."""
        k = self.d_qk // 2 + 4 * (self.d_qk // GROUP)
        v = 0 if self.v_aliases_k else self.d_v // 2 + 4 * (self.d_v // GROUP)
        return self.n_kv_heads * (k + v)

    def block_bytes(self):
        return BLOCK_TOKENS * self.row_bytes()

    def packed_bytes(self, n_tokens):
        """Whole blocks are persisted: L * ceil(n/256) * block bytes."""
        return self.n_layers * (-(-n_tokens // BLOCK_TOKENS)) * self.block_bytes()


class Pool:
    """A pool of physical blocks, kept tensor by tensor in the persisted schema.

    Per layer l and physical block b (Appendix A, groups along head_dim):
        Kc [Hkv][256][D/8] uint32, Ks/Kb [Hkv][256][D/64] float16,
        Vc [Hkv][256][Dv/8] uint32, Vs/Vb [Hkv][256][Dv/64] float16 (absent when V aliases K).
    With bfloat16 scales and biases (sb_dtype 1) the four 16-bit arrays are uint16 bit patterns.
    """

    def __init__(self, spec: Spec, n_blocks: int, fill: int = 0):
        s, T = spec, BLOCK_TOKENS
        self.spec, self.n_blocks = spec, n_blocks
        L, H = s.n_layers, s.n_kv_heads
        sb = np.float16 if s.sb_dtype == 0 else np.uint16
        self.Kc = np.full((L, n_blocks, H, T, s.d_qk // 8), fill, dtype=np.uint32)
        self.Ks = np.zeros((L, n_blocks, H, T, s.d_qk // GROUP), dtype=sb)
        self.Kb = np.zeros((L, n_blocks, H, T, s.d_qk // GROUP), dtype=sb)
        if not s.v_aliases_k:
            self.Vc = np.full((L, n_blocks, H, T, s.d_v // 8), fill, dtype=np.uint32)
            self.Vs = np.zeros((L, n_blocks, H, T, s.d_v // GROUP), dtype=sb)
            self.Vb = np.zeros((L, n_blocks, H, T, s.d_v // GROUP), dtype=sb)

    def tensors(self):
        t = [self.Kc, self.Ks, self.Kb]
        if not self.spec.v_aliases_k:
            t += [self.Vc, self.Vs, self.Vb]
        return t


def quantize_append(pool: Pool, layer, block_tables, pos, new_offs, k_new32, v_new32=None):
    """Quantize new K/V rows and write them at cache positions [pos[a], pos[a]+n_a).

    The 'update' half of update-and-fetch (Section 3.4), addressed through the
    per-agent block table (Section 3.1).  k_new32: [total_new][Hkv][D] float32
    (exact images of the bf16 inputs); v_new32 likewise, None when V aliases K.
    """
    s = pool.spec
    A = len(pos)
    kc, ks, kb = quantize_rows(k_new32, s.sb_dtype)
    kw = pack_codes(kc)
    if not s.v_aliases_k:
        vc, vs, vb = quantize_rows(v_new32, s.sb_dtype)
        vw = pack_codes(vc)
    for a in range(A):
        for i, row in enumerate(range(new_offs[a], new_offs[a + 1])):
            j = int(pos[a]) + i
            b = int(block_tables[a][j // BLOCK_TOKENS])
            assert 0 <= b < pool.n_blocks
            slot = j % BLOCK_TOKENS
            pool.Kc[layer, b, :, slot] = kw[row]
            pool.Ks[layer, b, :, slot] = ks[row]
            pool.Kb[layer, b, :, slot] = kb[row]
            if not s.v_aliases_k:
                pool.Vc[layer, b, :, slot] = vw[row]
                pool.Vs[layer, b, :, slot] = vs[row]
                pool.Vb[layer, b, :, slot] = vb[row]


def gather_dequant(pool: Pool, layer, table_row, lo, hi, kv_head):
    """Dequantized K [hi-lo][D] and V [hi-lo][Dv] (float64) of logical tokens lo..hi-1."""
    s = pool.spec
    j = np.arange(lo, hi)
    blk = np.asarray(table_row)[j // BLOCK_TOKENS]
    assert np.all((blk >= 0) & (blk < pool.n_blocks))
    slot = j % BLOCK_TOKENS
    K = dequantize(unpack_codes(pool.Kc[layer, blk, kv_head, slot]),
                   pool.Ks[layer, blk, kv_head, slot], pool.Kb[layer, blk, kv_head, slot])
    if s.v_aliases_k:
        V = K[:, : s.d_v]
    else:
        V = dequantize(unpack_codes(pool.Vc[layer, blk, kv_head, slot]),
                       pool.Vs[layer, blk, kv_head, slot], pool.Vb[layer, blk, kv_head, slot])
    return K, V


# ----------------------------------------------------------------------------
# attention: the plain definition, float64
# ----------------------------------------------------------------------------
def _attend_one(q64, K, V, softmax_scale):
    """softmax(scale * K q) . V for one query vector; returns (out [Dv], lse)."""
    if K.shape[0] == 0:
        return np.zeros(V.shape[1], dtype=np.float64), -np.inf
    logits = softmax_scale * (K @ q64)
    m = logits.max()
    e = np.exp(logits - m)
    ssum = e.sum()
    p = e / ssum
    return p @ V, m + np.log(ssum)


def decode_attention(pool: Pool, layer, block_tables, kv_lens, window, q32, softmax_scale):
    """One query token per agent at position kv_len-1 over the whole Q4 cache.

    q32: [A][Hq][D] float32 (exact images of bf16).  Query head h reads KV head
    h // n_rep (Section 3.6).  window = 0: all keys; else the last `window` keys
    (the query itself and the window-1 tokens before it).
    Returns out [A][Hq][Dv] float64 and lse [A][Hq] float64 (natural log).
    """
    s = pool.spec
    A = len(kv_lens)
    out = np.zeros((A, s.n_q_heads, s.d_v), dtype=np.float64)
    lse = np.full((A, s.n_q_heads), -np.inf, dtype=np.float64)
    for a in range(A):
        n = int(kv_lens[a])
        lo = max(0, n - window) if window > 0 else 0
        for hk in range(s.n_kv_heads):
            K, V = gather_dequant(pool, layer, block_tables[a], lo, n, hk)
            for r in range(s.n_rep):
                h = hk * s.n_rep + r
                out[a, h], lse[a, h] = _attend_one(q32[a, h].astype(np.float64), K, V, softmax_scale)
    return out, lse


def prefill_attention(pool: Pool, layer, block_tables, kv_lens, q_offs, window, q32, softmax_scale,
                      rows=None):
    """Chunked-prefill attention (Sections 3.4, 3.5).

    Agent a's q_len = q_offs[a+1]-q_offs[a] new queries sit at positions
    kv_len-q_len+i; query i attends keys j <= position (and j > position-window
    when window > 0), all read from the Q4 cache (the new chunk was appended
    before this call).  q32: [total_q][Hq][D] float32.
    rows: optional iterable of global query rows to compute (others left zero).
    Returns out [total_q][Hq][Dv] float64 and lse [total_q][Hq].
    """
    s = pool.spec
    A = len(kv_lens)
    total_q = int(q_offs[A])
    out = np.zeros((total_q, s.n_q_heads, s.d_v), dtype=np.float64)
    lse = np.full((total_q, s.n_q_heads), -np.inf, dtype=np.float64)
    want = None if rows is None else set(int(r) for r in rows)
    for a in range(A):
        n = int(kv_lens[a])
        q_len = int(q_offs[a + 1] - q_offs[a])
        agent_rows = [i for i in range(q_len) if want is None or (int(q_offs[a]) + i) in want]
        if not agent_rows:
            continue
        for hk in range(s.n_kv_heads):
            K, V = gather_dequant(pool, layer, block_tables[a], 0, n, hk)
            for i in agent_rows:
                p = n - q_len + i
                lo = max(0, p + 1 - window) if window > 0 else 0
                row = int(q_offs[a]) + i
                for r in range(s.n_rep):
                    h = hk * s.n_rep + r
                    out[row, h], lse[row, h] = _attend_one(
                        q32[row, h].astype(np.float64), K[lo:p + 1], V[lo:p + 1], softmax_scale)
    return out, lse


# ----------------------------------------------------------------------------
# persisted layout (Appendix A): pack / unpack
# ----------------------------------------------------------------------------
def pack(pool: Pool, table_row, n_tokens) -> np.ndarray:
    """One agent's blocks, all layers, as one contiguous byte buffer.

    Order: layer outermost, then logical block, then the tensors
    K_codes | K_scales | K_biases | V_codes | V_scales | V_biases, each
    [Hkv][256][...] row-major.  Slots at or beyond n_tokens are zero bytes.
    """
    s = pool.spec
    nblk = -(-n_tokens // BLOCK_TOKENS)
    parts = []
    for l in range(s.n_layers):
        for lb in range(nblk):
            b = int(table_row[lb])
            assert 0 <= b < pool.n_blocks
            valid = min(BLOCK_TOKENS, n_tokens - lb * BLOCK_TOKENS)
            for t in pool.tensors():
                x = t[l, b].copy()
                x[:, valid:] = 0
                parts.append(x.reshape(-1).view(np.uint8))
    buf = np.concatenate(parts) if parts else np.zeros(0, dtype=np.uint8)
    assert buf.size == s.packed_bytes(n_tokens)
    return buf


def unpack(pool: Pool, table_row, n_tokens, buf: np.ndarray):
    """Inverse of pack: scatter a persisted buffer into the blocks named by table_row."""
    s = pool.spec
    buf = np.asarray(buf, dtype=np.uint8)
    assert buf.size == s.packed_bytes(n_tokens)
    nblk = -(-n_tokens // BLOCK_TOKENS)
    off = 0
    for l in range(s.n_layers):
        for lb in range(nblk):
            b = int(table_row[lb])
            assert 0 <= b < pool.n_blocks
            for t in pool.tensors():
                nbytes = t[l, b].nbytes
                t[l, b] = buf[off:off + nbytes].view(t.dtype).reshape(t[l, b].shape)
                off += nbytes


# ----------------------------------------------------------------------------
# persisted container (Appendix "safetensors Q4 Format")
# ----------------------------------------------------------------------------
def container_header(spec: Spec, n_tokens: int) -> bytes:
    """Header of the safetensors file that holds one agent's cache: 8-byte little-endian length, then JSON.

    Tensors are listed layer by layer and block by block under the paper's names
    L{l}_B{b}_{K,V}_{weights,scales,biases}, in the order of the data section
    (K codes, K scales, K biases, V codes, V scales, V biases), each with dtype,
    shape [Hkv][256][...] and byte range; "__metadata__" carries the spec and the
    token count as strings.  No blanks inside; padded with spaces so that the
    data section starts at a multiple of 64 bytes.
    """
    s, T, H = spec, BLOCK_TOKENS, spec.n_kv_heads
    nblk = -(-n_tokens // T)
    meta = [("format", "q4kv-1"), ("n_layers", s.n_layers), ("n_q_heads", s.n_q_heads), ("n_kv_heads", s.n_kv_heads),
            ("d_qk", s.d_qk), ("d_v", s.d_v), ("v_aliases_k", int(s.v_aliases_k)), ("group", GROUP),
            ("block_tokens", T), ("sb_dtype", s.sb_dtype), ("n_tokens", n_tokens)]
    parts = ['"__metadata__":{' + ",".join(f'"{k}":"{v}"' for k, v in meta) + "}"]
    off = 0
    sbt = "F16" if s.sb_dtype == 0 else "BF16"
    for l in range(s.n_layers):
        for b in range(nblk):
            tensors = [("K", "weights", "U32", s.d_qk // 8, 4), ("K", "scales", sbt, s.d_qk // GROUP, 2),
                       ("K", "biases", sbt, s.d_qk // GROUP, 2)]
            if not s.v_aliases_k:
                tensors += [("V", "weights", "U32", s.d_v // 8, 4), ("V", "scales", sbt, s.d_v // GROUP, 2),
                            ("V", "biases", sbt, s.d_v // GROUP, 2)]
            for kv, what, dt, last, esz in tensors:
                nb = H * T * last * esz
                parts.append(f'"L{l}_B{b}_{kv}_{what}":{{"dtype":"{dt}","shape":[{H},{T},{last}],'
                             f'"data_offsets":[{off},{off + nb}]}}')
                off += nb
    assert off == s.packed_bytes(n_tokens)
    js = ("{" + ",".join(parts) + "}").encode("ascii")
    total = (8 + len(js) + 63) // 64 * 64
    js = js + b" " * (total - 8 - len(js))
    return len(js).to_bytes(8, "little") + js


def container(pool: Pool, table_row, n_tokens) -> np.ndarray:
    """The whole file image of one agent: header, then the packed buffer."""
    head = np.frombuffer(container_header(pool.spec, n_tokens), dtype=np.uint8)
    return np.concatenate([head, pack(pool, table_row, n_tokens)])


# ----------------------------------------------------------------------------
# dense left-padded batch of one layer (Section 3.4: merge / extract)
# ----------------------------------------------------------------------------
def extract_dense(pool: Pool, layer, block_tables, kv_lens, T) -> np.ndarray:
    """The paper's merged cache of one layer as bytes: K codes [A][Hkv][T][D/8] u32, K scales, K biases
    [A][Hkv][T][D/64] f16, then the V tensors (absent when V aliases K), one after the other; agent a's
    tokens sit in rows T - len_a .. T - 1, the padding rows before them are zero."""
    s, A = pool.spec, len(kv_lens)
    outs = [np.zeros((A,) + t.shape[2:3] + (T,) + t.shape[4:], dtype=t.dtype) for t in pool.tensors()]
    for a, n in enumerate(kv_lens):
        assert 0 <= n <= T
        for j in range(n):
            b, slot = int(block_tables[a][j // BLOCK_TOKENS]), j % BLOCK_TOKENS
            for o, t in zip(outs, pool.tensors()):
                o[a, :, T - n + j] = t[layer, b, :, slot]
    return np.concatenate([o.reshape(-1).view(np.uint8) for o in outs])


def merge_dense(pool: Pool, layer, block_tables, kv_lens, T, dense: np.ndarray):
    """Inverse of extract_dense: the rows of a dense left-padded batch go to cache positions 0 .. len_a - 1."""
    s, A = pool.spec, len(kv_lens)
    dense = np.asarray(dense, dtype=np.uint8)
    off = 0
    for t in pool.tensors():
        shape = (A,) + t.shape[2:3] + (T,) + t.shape[4:]
        nb = int(np.prod(shape)) * t.dtype.itemsize
        d = dense[off:off + nb].view(t.dtype).reshape(shape)
        off += nb
        for a, n in enumerate(kv_lens):
            for j in range(n):
                b, slot = int(block_tables[a][j // BLOCK_TOKENS]), j % BLOCK_TOKENS
                t[layer, b, :, slot] = d[a, :, T - n + j]
    assert off == dense.size

