"""The persisted container (Appendix "safetensors Q4 Format"): the oracle's file image is pinned with the safetensors
package (an independent reader), the library's host-side header writer must produce the same bytes, and its reader must
take them back.  No kernel is launched here."""
import json

import numpy as np
import pytest

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import binding as B, synth


def _pool_with_content(spec, n_blocks, seed):
    pool = O.Pool(spec, n_blocks)
    g = synth.rng(seed, 0)
    for t in pool.tensors():
        if t.dtype == np.uint32:
            t[:] = g.integers(0, 2**32, size=t.shape, dtype=np.uint64).astype(np.uint32)
        else:
            t[:] = g.standard_normal(t.shape).astype(np.float16)
    return pool


@pytest.mark.parametrize("args,n_tokens", [((2, 8, 2, 128, 128, False), 300), ((1, 16, 1, 576, 512, True), 256),
                                           ((1, 4, 4, 192, 128, False), 17)])
def test_oracle_container_opens_with_the_safetensors_package(args, n_tokens):
    safetensors_numpy = pytest.importorskip("safetensors.numpy")
    spec = O.Spec(*args)
    nblk = -(-n_tokens // 256)
    pool = _pool_with_content(spec, nblk + 2, 5)
    row = list(range(nblk + 1, 1, -1))[:nblk]                 # logical block b sits in physical block row[b]
    image = O.container(pool, row, n_tokens).tobytes()
    tensors = safetensors_numpy.load(image)
    expect = 6 if not spec.v_aliases_k else 3
    assert len(tensors) == spec.n_layers * nblk * expect
    H = spec.n_kv_heads
    for l in range(spec.n_layers):
        for b in range(nblk):
            valid = min(256, n_tokens - 256 * b)
            pairs = [("K_weights", pool.Kc, np.uint32, spec.d_qk // 8), ("K_scales", pool.Ks, np.float16, spec.d_qk // 64),
                     ("K_biases", pool.Kb, np.float16, spec.d_qk // 64)]
            if not spec.v_aliases_k:
                pairs += [("V_weights", pool.Vc, np.uint32, spec.d_v // 8), ("V_scales", pool.Vs, np.float16, spec.d_v // 64),
                          ("V_biases", pool.Vb, np.float16, spec.d_v // 64)]
            for name, src, dt, last in pairs:
                t = tensors[f"L{l}_B{b}_{name}"]
                assert t.dtype == dt and t.shape == (H, 256, last)
                want = src[l, row[b]].copy()
                want[:, valid:] = 0                                   # slots past the cache end are zero bytes
                assert np.array_equal(t.view(np.uint8), want.view(np.uint8)), name
    # the header itself: length prefix, metadata strings, data section = the packed buffer
    n = int.from_bytes(image[:8], "little")
    head = json.loads(image[8:8 + n])
    assert (8 + n) % 64 == 0
    assert head["__metadata__"]["n_tokens"] == str(n_tokens) and head["__metadata__"]["d_qk"] == str(spec.d_qk)
    assert head["L0_B0_K_weights"]["data_offsets"][0] == 0
    assert np.array_equal(np.frombuffer(image[8 + n:], dtype=np.uint8), O.pack(pool, row, n_tokens))


@pytest.mark.parametrize("args,n_tokens", [((32, 32, 8, 128, 128, False), 4096), ((2, 8, 2, 128, 128, False), 300),
                                           ((27, 16, 1, 576, 512, True), 1000), ((1, 4, 4, 192, 128, False), 1)])
@pytest.mark.parametrize("sb_dtype", [0, 1])
def test_library_header_equals_the_oracles_and_reads_back(args, n_tokens, sb_dtype):
    ospec = O.Spec(*args, sb_dtype=sb_dtype)
    spec = B.Spec.make(*args, sb_dtype=sb_dtype)
    want = O.container_header(ospec, n_tokens)
    got = B.q4kv_container_write_header(spec, n_tokens)
    assert B.q4kv_container_header_bytes(spec, n_tokens) == len(want)
    assert got == want
    back, nt, off = B.q4kv_container_read_header(want)
    assert nt == n_tokens and off == len(want)
    assert (back.n_layers, back.n_q_heads, back.n_kv_heads, back.d_qk, back.d_v, back.v_aliases_k, back.sb_dtype) == \
        (args[0], args[1], args[2], args[3], args[4], int(args[5]), sb_dtype)
    # a header that is not this library's canonical text is refused
    bad = bytearray(want)
    i = bad.index(b'"L0_B0_K_weights"')
    bad[i + 2] = ord("9")
    with pytest.raises(B.Q4KVError):
        B.q4kv_container_read_header(bytes(bad))
    with pytest.raises(B.Q4KVError):
        B.q4kv_container_read_header(want[:40])
