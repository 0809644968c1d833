"""The allocation-free decode entry point against the ordinary one.

`q4kv_decode_attention_static` serves hosts that cannot allocate device memory at call time (all of
their memory was handed out at start-up, or the pool is not theirs to touch): it keeps the split
partials in a fixed array inside the library instead of a caller workspace.  It must return what
`q4kv_decode_attention` returns, call after call, although every call reuses the same array and
finds the previous call's leftovers in it.  This file sorts last on purpose, so a run that stops at
the first failure has already run everything else; it also passes when run alone in a fresh process
(the first call then does the per-device set-up).
"""
import math

import numpy as np
import pytest
import torch

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import synth

pytestmark = pytest.mark.gpu

ATOL, RTOL_ROW = 2e-3, 1e-2


def _close(got, ref):
    got = got.double().cpu().numpy()
    ref = ref.double().cpu().numpy()
    err = np.abs(got - ref)
    assert np.all(np.isfinite(got))
    assert err.max() <= ATOL
    rows = err.reshape(-1, ref.shape[-1]).max(axis=1)
    mags = np.abs(ref).reshape(-1, ref.shape[-1]).max(axis=1)
    assert np.all(rows <= RTOL_ROW * mags + 1e-30)


def test_static_scratch_entry_matches_workspace_entry_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_04428_b200 import binding as B, harness as H

    L, Hq, Hkv, D = 1, 8, 2, 128
    scale = 1.0 / math.sqrt(D)
    # two different batches, so the second call finds partials of another shape left in the array
    cases = [([1000, 700, 33], 0, 11), ([300, 1500], 256, 12)]
    for lens, window, seed in cases:
        dc, opool, tabs = _filled_cache(H, (L, Hq, Hkv, D, D, False), lens, seed)
        q_bits = synth.normal_bf16(seed, 7, (len(lens), Hq, D))
        q = H.bf16_dev(q_bits)
        lens_d = H.dev(np.asarray(lens, dtype=np.int32))
        ref, ref_lse = dc.decode(0, lens_d, window, q, scale)          # caller-supplied workspace
        oref, _ = O.decode_attention(opool, 0, tabs, lens, window, synth.bf16_bits_to_f32(q_bits), scale)
        for _ in range(2):                                               # two calls in a row
            out = torch.full_like(ref, float("nan"))
            lse = torch.full_like(ref_lse, float("nan"))
            B.q4kv_decode_attention_static(dc.spec, dc.pool, dc.n_blocks, 0, dc.bt, lens_d, 0, window, q, scale,
                                           out, B.OUT_F32, lse, dc.flags)
            torch.cuda.synchronize()
            _close(out, ref)
            _close(out, torch.from_numpy(oref))
            assert torch.allclose(lse, ref_lse, rtol=0, atol=2e-3)
        assert dc.read_flags() == 0


def _filled_cache(H, spec_args, lens, seed):
    """The same tokens in a device cache and in an oracle pool."""
    L, Hq, Hkv, D, Dv, alias = spec_args
    n_blocks = sum(-(-n // 256) for n in lens) + 2
    tabs = synth.block_tables(seed, 99, lens, n_blocks)
    dc = H.DeviceCache(L, Hq, Hkv, D, Dv, alias, n_blocks, tabs)
    opool = O.Pool(O.Spec(L, Hq, Hkv, D, Dv, alias), n_blocks)
    f32 = synth.bf16_bits_to_f32
    for a, n in enumerate(lens):
        k = synth.kv_bf16(seed, 10 * a + 1, n, Hkv, D)
        v = None if alias else synth.kv_bf16(seed, 10 * a + 2, n, Hkv, Dv)
        _, bt = dc.sub_batch(a, a + 1)
        dc.append(0, [0], [0, n], k, v, bt=bt)
        O.quantize_append(opool, 0, tabs[a:a + 1], [0], [0, n], f32(k), None if v is None else f32(v))
    return dc, opool, tabs


def test_static_scratch_entry_across_kernels_and_growing_batches():
    """Every call shares the one array, whatever kernel serves it: a latent-cache call (its own kernel), a d = 192 call
    (the shape-agnostic kernel) and a 2-agent call each leave their partial records in it, and the call that follows --
    a GQA batch of 10 agents x 8 KV heads, whose arrival counters reach further into the array than any of theirs --
    must still return what q4kv_decode_attention returns on a fresh zero-filled workspace, and what the oracle
    returns.  Outputs start as NaN so that a row nobody wrote is seen."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_04428_b200 import binding as B, harness as H

    gqa = (1, 32, 8, 128, 128, False)
    big_lens = [700, 300, 260, 5000, 90, 1200, 64, 33, 2000, 513]
    calls = [
        ((1, 16, 1, 576, 512, True), [600, 70], 1.0 / math.sqrt(192), 21),
        (gqa, big_lens, 1.0 / math.sqrt(128), 22),
        ((1, 4, 4, 192, 128, False), [400, 300], 1.0 / math.sqrt(192), 23),
        (gqa, big_lens, 1.0 / math.sqrt(128), 22),
        (gqa, [900, 40], 1.0 / math.sqrt(128), 24),
        (gqa, big_lens, 1.0 / math.sqrt(128), 22),
    ]
    caches = {}
    for spec_args, lens, scale, seed in calls:
        if seed not in caches:
            caches[seed] = _filled_cache(H, spec_args, lens, seed)
        dc, opool, tabs = caches[seed]
        q_bits = synth.normal_bf16(seed, 7, (len(lens), spec_args[1], spec_args[3]))
        q = H.bf16_dev(q_bits)
        lens_d = H.dev(np.asarray(lens, dtype=np.int32))
        dc._ws = None                                                    # a fresh, zero-filled workspace for the comparand
        ref, ref_lse = dc.decode(0, lens_d, 0, q, scale)
        oref, _ = O.decode_attention(opool, 0, tabs, lens, 0, synth.bf16_bits_to_f32(q_bits), scale)
        out = torch.full_like(ref, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        B.q4kv_decode_attention_static(dc.spec, dc.pool, dc.n_blocks, 0, dc.bt, lens_d, 0, 0, q, scale,
                                       out, B.OUT_F32, lse, dc.flags)
        torch.cuda.synchronize()
        _close(out, ref)
        _close(out, torch.from_numpy(oref))
        assert torch.allclose(lse, ref_lse, rtol=0, atol=2e-3)
        assert dc.read_flags() == 0


def test_static_scratch_entry_rejects_batches_beyond_its_fixed_array():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2603_04428_b200 import binding as B, harness as H

    # thousands of agents need more partial records than the fixed array holds
    A = 4096
    spec = B.Spec.make(1, 32, 8, 128, 128)
    assert B.q4kv_workspace_bytes(spec, A, 256, 0) > B.STATIC_SCRATCH_BYTES
    tabs = H.dev(np.zeros((A, 1), dtype=np.int32))
    dummy = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.Q4KVError) as e:
        B.q4kv_decode_attention_static(spec, dummy, 1, 0, B.batch(tabs), dummy, 256, 0, dummy, 0.1, dummy, B.OUT_F32,
                                       None, None)
    assert e.value.code == B.EWORKSPACE
