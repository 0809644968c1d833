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
        n_blocks = sum(-(-n // 256) for n in lens) + 2
        tabs = synth.block_tables(seed, 99, lens, n_blocks)
        dc = H.DeviceCache(L, Hq, Hkv, D, D, False, n_blocks, tabs)
        for a, n in enumerate(lens):
            _, bt = dc.sub_batch(a, a + 1)
            dc.append(0, [0], [0, n], synth.kv_bf16(seed, 10 * a + 1, n, Hkv, D),
                      synth.kv_bf16(seed, 10 * a + 2, n, Hkv, D), bt=bt)
        q = H.bf16_dev(synth.normal_bf16(seed, 7, (len(lens), Hq, D)))
        lens_d = H.dev(np.asarray(lens, dtype=np.int32))
        ref, ref_lse = dc.decode(0, lens_d, window, q, scale)          # caller-supplied workspace
        for _ in range(2):                                               # two calls in a row
            out = torch.full_like(ref, float("nan"))
            lse = torch.full_like(ref_lse, float("nan"))
            B.q4kv_decode_attention_static(dc.spec, dc.pool, dc.n_blocks, 0, dc.bt, lens_d, 0, window, q, scale,
                                           out, B.OUT_F32, lse, dc.flags)
            torch.cuda.synchronize()
            _close(out, ref)
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
