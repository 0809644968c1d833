"""Host-side block bookkeeping (Section 3.1: per-agent isolation, LRU eviction) and the oracle's dense-batch
functions (Section 3.4: merge / extract).  No kernel is launched here."""
import numpy as np
import pytest

from oracle import q4kv_oracle as O
from paper_2603_04428_b200 import binding as B, synth


def test_blocks_are_exclusive_grow_in_place_and_come_back_on_release():
    al = B.Allocator(10)
    r1 = al.reserve(101, 300, 6)
    assert r1[:2] == [0, 1] and r1[2:] == [-1] * 4 and al.free_blocks() == 8
    r2 = al.reserve(202, 1024, 6)
    assert len(set(r2[:4]) & set(r1[:2])) == 0 and al.free_blocks() == 4          # isolation: no shared block
    r1b = al.reserve(101, 700, 6)                                                    # growth keeps the earlier blocks
    assert r1b[:2] == r1[:2] and r1b[2] not in r2[:4] and al.agent_blocks(101) == 3
    assert al.reserve(101, 100, 6)[:3] == r1b[:3]                                    # never shrinks
    with pytest.raises(B.Q4KVError) as e:
        al.reserve(303, 256 * 4, 6)                                                  # 3 free blocks only
    assert e.value.code == B.EWORKSPACE and al.agent_blocks(303) == 0
    with pytest.raises(B.Q4KVError):
        al.reserve(303, 256 * 7, 6)                                                  # more than a table row holds
    al.release(202)
    assert al.free_blocks() == 7 and al.agent_blocks(202) == 0
    r3 = al.reserve(303, 256 * 4, 6)
    assert set(r3[:4]).isdisjoint(r1b[:3])
    al.close()


def test_victims_come_in_least_recently_used_order_and_pinned_agents_are_spared():
    al = B.Allocator(6)
    for agent in (1, 2, 3):
        al.reserve(agent, 512, 2)
    assert al.free_blocks() == 0
    assert al.pick_victim() == 1
    al.touch(1)                                     # 1 was just used: 2 is now the oldest
    assert al.pick_victim() == 2
    al.pin(2, True)
    assert al.pick_victim() == 3
    al.reserve(3, 512, 2)                           # a reserve counts as a use
    assert al.pick_victim() == 1
    al.pin(1, True); al.pin(3, True)
    with pytest.raises(B.Q4KVError) as e:
        al.pick_victim()
    assert e.value.code == B.EWORKSPACE
    al.pin(2, False)
    v = al.pick_victim()
    assert v == 2
    al.release(v)                                   # the caller persisted it first
    assert al.reserve(4, 300, 2)[:2] != [-1, -1] and al.free_blocks() == 0
    with pytest.raises(B.Q4KVError):
        al.touch(2)                                 # released agents are forgotten
    al.close()


def test_oracle_dense_batch_is_left_padded_and_merge_inverts_extract():
    spec = O.Spec(2, 4, 2, 128, 64)
    lens, n_blocks, T = [300, 5, 0, 256], 6, 320
    tabs = synth.block_tables(7, 1, lens, n_blocks)
    pool = O.Pool(spec, n_blocks)
    g = synth.rng(7, 2)
    for t in pool.tensors():
        t[:] = g.integers(1, 200, size=t.shape).astype(t.dtype)                     # no zero anywhere
    dense = O.extract_dense(pool, 1, tabs, lens, T)
    A, H = len(lens), spec.n_kv_heads
    assert dense.size == B.q4kv_dense_bytes(B.Spec.make(2, 4, 2, 128, 64), A, T) == A * H * T * (64 + 8 + 32 + 4)
    kc = dense[:A * H * T * 64].view(np.uint32).reshape(A, H, T, 16)
    ks = dense[A * H * T * 64:A * H * T * 68].view(np.float16).reshape(A, H, T, 2)
    assert np.all(kc[0, :, :T - 300] == 0) and np.all(kc[2] == 0) and np.all(kc[1, :, :T - 5] == 0)   # left padding
    # literal positions: agent 0, head 1, cache position 299 (block 1, slot 43) is the last row; position 0 is row T - 300
    assert np.array_equal(kc[0, 1, T - 1], pool.Kc[1, tabs[0][1], 1, 43]) and np.array_equal(kc[0, 1, T - 300], pool.Kc[1, tabs[0][0], 1, 0])
    assert np.array_equal(ks[3, 0, T - 256], pool.Ks[1, tabs[3][0], 0, 0])
    pool2 = O.Pool(spec, n_blocks)
    tabs2 = synth.block_tables(8, 1, lens, n_blocks)
    O.merge_dense(pool2, 1, tabs2, lens, T, dense)
    assert np.array_equal(O.extract_dense(pool2, 1, tabs2, lens, T), dense)
    assert np.all(pool2.Kc[0] == 0)                                                  # the other layer is untouched
