"""Thin ctypes binding of libq4kv.so: argument marshalling only.

Every function has the name and argument order of its C entry point
(include/q4kv.h).  Tensors are torch CUDA tensors used purely as device
memory; the current torch CUDA stream is passed as the stream.  There is no
CPU path: loading fails loudly when the library has not been built, and every
call raises Q4KVError on a negative status.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libq4kv.so")

OK, EINVAL, EUNSUPPORTED, EWORKSPACE, ECUDA = 0, -1, -2, -3, -4
FLAG_BAD_BLOCK, FLAG_BAD_LENGTH, FLAG_INTERNAL, FLAG_SB_RANGE = 1, 2, 4, 8
OUT_F32, OUT_BF16 = 0, 1

EXPORTS = [
    "q4kv_status_string", "q4kv_pool_bytes", "q4kv_packed_bytes", "q4kv_workspace_bytes",
    "q4kv_quantize_append", "q4kv_decode_attention", "q4kv_prefill_attention", "q4kv_pack", "q4kv_unpack",
    "q4kv_decode_attention_static", "q4kv_append_decode_attention", "q4kv_decode_attention_layers",
    "q4kv_workspace_bytes_layers",
    "q4kv_container_header_bytes", "q4kv_container_write_header", "q4kv_container_read_header", "q4kv_save", "q4kv_restore",
    "q4kv_allocator_create", "q4kv_allocator_destroy", "q4kv_allocator_free_blocks", "q4kv_allocator_agent_blocks",
    "q4kv_allocator_reserve", "q4kv_allocator_touch", "q4kv_allocator_pin", "q4kv_allocator_pick_victim",
    "q4kv_allocator_release", "q4kv_dense_bytes", "q4kv_merge_dense", "q4kv_extract_dense",
]
STATIC_SCRATCH_BYTES = 8 << 20
WORKSPACE_HEADER_BYTES = 65536


class Q4KVError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class Spec(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "d_qk", "d_v", "v_aliases_k", "group", "block_tokens", "sb_dtype",
        "exact_products")]

    @classmethod
    def make(cls, n_layers, n_q_heads, n_kv_heads, d_qk, d_v, v_aliases_k=False, exact_products=False, sb_dtype=0):
        return cls(n_layers, n_q_heads, n_kv_heads, d_qk, d_v, int(bool(v_aliases_k)), 64, 256, int(sb_dtype),
                   int(bool(exact_products)))


class Batch(ctypes.Structure):
    _fields_ = [("n_agents", ctypes.c_int32), ("max_blocks", ctypes.c_int32), ("block_tables", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2603_04428_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
        sp, bp = ctypes.POINTER(Spec), ctypes.POINTER(Batch)
        L.q4kv_status_string.restype = ctypes.c_char_p
        L.q4kv_status_string.argtypes = [ctypes.c_int]
        L.q4kv_pool_bytes.restype = sz
        L.q4kv_pool_bytes.argtypes = [sp, i32]
        L.q4kv_packed_bytes.restype = sz
        L.q4kv_packed_bytes.argtypes = [sp, i32]
        L.q4kv_workspace_bytes.restype = sz
        L.q4kv_workspace_bytes.argtypes = [sp, i32, i32, i32]
        L.q4kv_quantize_append.restype = ctypes.c_int
        L.q4kv_quantize_append.argtypes = [sp, vp, i32, i32, bp, vp, vp, i32, vp, vp, vp, vp]
        L.q4kv_decode_attention.restype = ctypes.c_int
        L.q4kv_decode_attention.argtypes = [sp, vp, i32, i32, bp, vp, i32, i32, vp, f32, vp, i32, vp, vp, sz, vp, vp]
        L.q4kv_append_decode_attention.restype = ctypes.c_int
        L.q4kv_append_decode_attention.argtypes = [sp, vp, i32, i32, bp, vp, i32, i32, vp, vp, vp, f32, vp, i32, vp, vp,
                                                   sz, vp, vp]
        L.q4kv_workspace_bytes_layers.restype = sz
        L.q4kv_workspace_bytes_layers.argtypes = [sp, i32, i32, i32]
        L.q4kv_decode_attention_layers.restype = ctypes.c_int
        L.q4kv_decode_attention_layers.argtypes = [sp, vp, i32, i32, i32, bp, vp, i32, ctypes.POINTER(i32), vp, vp, vp, f32, vp,
                                                   i32, vp, vp, sz, vp, vp]
        L.q4kv_decode_attention_static.restype = ctypes.c_int
        L.q4kv_decode_attention_static.argtypes = [sp, vp, i32, i32, bp, vp, i32, i32, vp, f32, vp, i32, vp, vp, vp]
        L.q4kv_prefill_attention.restype = ctypes.c_int
        L.q4kv_prefill_attention.argtypes = [sp, vp, i32, i32, bp, vp, vp, i32, i32, i32, i32, vp, f32, vp, i32, vp,
                                             vp, sz, vp, vp]
        L.q4kv_container_header_bytes.restype = sz
        L.q4kv_container_header_bytes.argtypes = [sp, i32]
        L.q4kv_container_write_header.restype = ctypes.c_int
        L.q4kv_container_write_header.argtypes = [sp, i32, vp, sz]
        L.q4kv_container_read_header.restype = ctypes.c_int
        L.q4kv_container_read_header.argtypes = [vp, sz, sp, ctypes.POINTER(i32), ctypes.POINTER(sz)]
        L.q4kv_save.restype = ctypes.c_int
        L.q4kv_save.argtypes = [sp, vp, i32, vp, i32, vp, sz, vp, sz, vp, vp]
        L.q4kv_restore.restype = ctypes.c_int
        L.q4kv_restore.argtypes = [sp, vp, sz, i32, vp, i32, vp, vp, sz, vp, vp, vp]
        i64 = ctypes.c_int64
        L.q4kv_allocator_create.restype = vp
        L.q4kv_allocator_create.argtypes = [i32]
        L.q4kv_allocator_destroy.restype = None
        L.q4kv_allocator_destroy.argtypes = [vp]
        L.q4kv_allocator_free_blocks.restype = i32
        L.q4kv_allocator_free_blocks.argtypes = [vp]
        L.q4kv_allocator_agent_blocks.restype = i32
        L.q4kv_allocator_agent_blocks.argtypes = [vp, i64]
        L.q4kv_allocator_reserve.restype = ctypes.c_int
        L.q4kv_allocator_reserve.argtypes = [vp, i64, i32, ctypes.POINTER(i32), i32]
        L.q4kv_allocator_touch.restype = ctypes.c_int
        L.q4kv_allocator_touch.argtypes = [vp, i64]
        L.q4kv_allocator_pin.restype = ctypes.c_int
        L.q4kv_allocator_pin.argtypes = [vp, i64, i32]
        L.q4kv_allocator_pick_victim.restype = ctypes.c_int
        L.q4kv_allocator_pick_victim.argtypes = [vp, ctypes.POINTER(i64)]
        L.q4kv_allocator_release.restype = ctypes.c_int
        L.q4kv_allocator_release.argtypes = [vp, i64]
        L.q4kv_dense_bytes.restype = sz
        L.q4kv_dense_bytes.argtypes = [sp, i32, i32]
        L.q4kv_merge_dense.restype = ctypes.c_int
        L.q4kv_merge_dense.argtypes = [sp, vp, i32, i32, bp, vp, i32, vp, sz, vp, vp]
        L.q4kv_extract_dense.restype = ctypes.c_int
        L.q4kv_extract_dense.argtypes = [sp, vp, i32, i32, bp, vp, i32, vp, sz, vp, vp]
        L.q4kv_pack.restype = ctypes.c_int
        L.q4kv_pack.argtypes = [sp, vp, i32, vp, i32, vp, sz, vp, vp]
        L.q4kv_unpack.restype = ctypes.c_int
        L.q4kv_unpack.argtypes = [sp, vp, sz, i32, vp, i32, vp, vp, vp]
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "device pointers come from contiguous CUDA tensors"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(code, where):
    if code != OK:
        raise Q4KVError(code, where)


def status_string(code: int) -> str:
    return lib().q4kv_status_string(int(code)).decode()


def batch(block_tables: torch.Tensor) -> Batch:
    assert block_tables.dtype == torch.int32 and block_tables.dim() == 2
    return Batch(block_tables.shape[0], block_tables.shape[1], _ptr(block_tables))


def q4kv_pool_bytes(spec: Spec, n_blocks: int) -> int:
    return lib().q4kv_pool_bytes(ctypes.byref(spec), n_blocks)


def q4kv_packed_bytes(spec: Spec, n_tokens: int) -> int:
    return lib().q4kv_packed_bytes(ctypes.byref(spec), n_tokens)


def q4kv_workspace_bytes(spec: Spec, n_agents: int, max_kv_len: int, total_q: int) -> int:
    return lib().q4kv_workspace_bytes(ctypes.byref(spec), n_agents, max_kv_len, total_q)


def q4kv_quantize_append(spec, pool, n_blocks, layer, bt: Batch, pos, new_offs, total_new, k_new, v_new,
                         status_flags=None):
    _check(lib().q4kv_quantize_append(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt), _ptr(pos),
                                      _ptr(new_offs), total_new, _ptr(k_new), _ptr(v_new), _ptr(status_flags),
                                      _stream()), "q4kv_quantize_append")


def q4kv_decode_attention(spec, pool, n_blocks, layer, bt: Batch, kv_lens, max_kv_len, window, q, softmax_scale,
                          out, out_dtype, lse, workspace, status_flags=None):
    _check(lib().q4kv_decode_attention(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt),
                                       _ptr(kv_lens), max_kv_len, window, _ptr(q), softmax_scale, _ptr(out),
                                       out_dtype, _ptr(lse), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream()),
           "q4kv_decode_attention")


def q4kv_append_decode_attention(spec, pool, n_blocks, layer, bt: Batch, kv_lens, max_kv_len, window, k_new, v_new, q,
                                 softmax_scale, out, out_dtype, lse, workspace, status_flags=None):
    """Update-and-fetch in one launch: quantize one new token per agent into the cache (position kv_len - 1) and
    attend over the cache including it."""
    _check(lib().q4kv_append_decode_attention(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt),
                                              _ptr(kv_lens), max_kv_len, window, _ptr(k_new), _ptr(v_new), _ptr(q),
                                              softmax_scale, _ptr(out), out_dtype, _ptr(lse), _ptr(workspace),
                                              workspace.numel() * workspace.element_size(), _ptr(status_flags),
                                              _stream()),
           "q4kv_append_decode_attention")


def q4kv_decode_attention_static(spec, pool, n_blocks, layer, bt: Batch, kv_lens, max_kv_len, window, q, softmax_scale,
                                 out, out_dtype, lse, status_flags=None):
    """Decode attention for callers that cannot hand over a workspace: the scratch is a fixed array inside the
    library (STATIC_SCRATCH_BYTES per GPU), so this call allocates nothing.  Calls that overlap on the GPU race."""
    _check(lib().q4kv_decode_attention_static(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt),
                                              _ptr(kv_lens), max_kv_len, window, _ptr(q), softmax_scale, _ptr(out),
                                              out_dtype, _ptr(lse), _ptr(status_flags), _stream()),
           "q4kv_decode_attention_static")


def q4kv_prefill_attention(spec, pool, n_blocks, layer, bt: Batch, kv_lens, q_offs, total_q, max_q_len, max_kv_len,
                           window, q, softmax_scale, out, out_dtype, lse, workspace, status_flags=None):
    _check(lib().q4kv_prefill_attention(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt),
                                        _ptr(kv_lens), _ptr(q_offs), total_q, max_q_len, max_kv_len, window, _ptr(q),
                                        softmax_scale, _ptr(out), out_dtype, _ptr(lse), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream()),
           "q4kv_prefill_attention")


def q4kv_pack(spec, pool, n_blocks, block_table_row, n_tokens, dst, status_flags=None):
    _check(lib().q4kv_pack(ctypes.byref(spec), _ptr(pool), n_blocks, _ptr(block_table_row), n_tokens, _ptr(dst),
                           dst.numel() * dst.element_size(), _ptr(status_flags), _stream()), "q4kv_pack")


def q4kv_unpack(spec, src, n_tokens, pool, n_blocks, block_table_row, status_flags=None):
    _check(lib().q4kv_unpack(ctypes.byref(spec), _ptr(src), src.numel() * src.element_size(), n_tokens, _ptr(pool),
                             n_blocks, _ptr(block_table_row), _ptr(status_flags), _stream()), "q4kv_unpack")


def q4kv_container_header_bytes(spec: Spec, n_tokens: int) -> int:
    return lib().q4kv_container_header_bytes(ctypes.byref(spec), n_tokens)


def q4kv_container_write_header(spec: Spec, n_tokens: int) -> bytes:
    """The container header (host only) as bytes."""
    n = q4kv_container_header_bytes(spec, n_tokens)
    buf = ctypes.create_string_buffer(n)
    _check(lib().q4kv_container_write_header(ctypes.byref(spec), n_tokens, buf, n), "q4kv_container_write_header")
    return buf.raw


def q4kv_container_read_header(data: bytes):
    """(spec, n_tokens, data_offset) of a container whose first bytes are `data` (host only)."""
    spec = Spec()
    nt, off = ctypes.c_int32(0), ctypes.c_size_t(0)
    buf = ctypes.create_string_buffer(bytes(data), len(data))
    _check(lib().q4kv_container_read_header(buf, len(data), ctypes.byref(spec), ctypes.byref(nt), ctypes.byref(off)),
           "q4kv_container_read_header")
    return spec, nt.value, off.value


def q4kv_save(spec, pool, n_blocks, block_table_row, n_tokens, dev_staging, host_image, status_flags=None):
    """host_image: a pinned CPU uint8 tensor; complete once the current stream has run."""
    assert not host_image.is_cuda and host_image.is_contiguous()
    _check(lib().q4kv_save(ctypes.byref(spec), _ptr(pool), n_blocks, _ptr(block_table_row), n_tokens, _ptr(dev_staging),
                           dev_staging.numel(), host_image.data_ptr(), host_image.numel(), _ptr(status_flags), _stream()),
           "q4kv_save")


def q4kv_restore(spec, host_packed, n_tokens, pool, n_blocks, block_table_row, dev_staging, status_flags=None,
                 copy_stream=None, unpack_stream=None):
    """host_packed: a pinned CPU uint8 tensor holding the container's data section."""
    assert not host_packed.is_cuda and host_packed.is_contiguous()
    cs = copy_stream.cuda_stream if copy_stream is not None else _stream()
    us = unpack_stream.cuda_stream if unpack_stream is not None else _stream()
    _check(lib().q4kv_restore(ctypes.byref(spec), host_packed.data_ptr(), host_packed.numel(), n_tokens, _ptr(pool), n_blocks,
                              _ptr(block_table_row), _ptr(dev_staging), dev_staging.numel(), _ptr(status_flags), cs, us),
           "q4kv_restore")


class Allocator:
    """Thin holder of a q4kv_allocator (host-side block bookkeeping with LRU order)."""

    def __init__(self, n_blocks: int):
        self._h = lib().q4kv_allocator_create(n_blocks)
        if not self._h:
            raise Q4KVError(EINVAL, "q4kv_allocator_create")

    def close(self):
        if self._h:
            lib().q4kv_allocator_destroy(self._h)
            self._h = None

    __del__ = close

    def free_blocks(self) -> int:
        return lib().q4kv_allocator_free_blocks(self._h)

    def agent_blocks(self, agent_id: int) -> int:
        return lib().q4kv_allocator_agent_blocks(self._h, agent_id)

    def reserve(self, agent_id: int, n_tokens: int, max_blocks: int):
        row = (ctypes.c_int32 * max_blocks)()
        _check(lib().q4kv_allocator_reserve(self._h, agent_id, n_tokens, row, max_blocks), "q4kv_allocator_reserve")
        return list(row)

    def touch(self, agent_id: int):
        _check(lib().q4kv_allocator_touch(self._h, agent_id), "q4kv_allocator_touch")

    def pin(self, agent_id: int, pinned: bool):
        _check(lib().q4kv_allocator_pin(self._h, agent_id, int(pinned)), "q4kv_allocator_pin")

    def pick_victim(self) -> int:
        v = ctypes.c_int64(0)
        _check(lib().q4kv_allocator_pick_victim(self._h, ctypes.byref(v)), "q4kv_allocator_pick_victim")
        return v.value

    def release(self, agent_id: int):
        _check(lib().q4kv_allocator_release(self._h, agent_id), "q4kv_allocator_release")


def q4kv_dense_bytes(spec: Spec, n_agents: int, T: int) -> int:
    return lib().q4kv_dense_bytes(ctypes.byref(spec), n_agents, T)


def q4kv_merge_dense(spec, pool, n_blocks, layer, bt: Batch, kv_lens, T, dense, status_flags=None):
    _check(lib().q4kv_merge_dense(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt), _ptr(kv_lens), T,
                                  _ptr(dense), dense.numel() * dense.element_size(), _ptr(status_flags), _stream()),
           "q4kv_merge_dense")


def q4kv_extract_dense(spec, pool, n_blocks, layer, bt: Batch, kv_lens, T, dense, status_flags=None):
    _check(lib().q4kv_extract_dense(ctypes.byref(spec), _ptr(pool), n_blocks, layer, ctypes.byref(bt), _ptr(kv_lens), T,
                                    _ptr(dense), dense.numel() * dense.element_size(), _ptr(status_flags), _stream()),
           "q4kv_extract_dense")


def q4kv_workspace_bytes_layers(spec: Spec, n_agents: int, max_kv_len: int, layer_count: int) -> int:
    return lib().q4kv_workspace_bytes_layers(ctypes.byref(spec), n_agents, max_kv_len, layer_count)


def q4kv_decode_attention_layers(spec, pool, n_blocks, layer_begin, layer_count, bt: Batch, kv_lens, max_kv_len, windows,
                                 k_new, v_new, q, softmax_scale, out, out_dtype, lse, workspace, status_flags=None):
    """Decode attention (k_new, v_new None) or update-and-fetch for layer_count layers in one launch; windows: a host list."""
    w = (ctypes.c_int32 * layer_count)(*[int(x) for x in windows])
    _check(lib().q4kv_decode_attention_layers(ctypes.byref(spec), _ptr(pool), n_blocks, layer_begin, layer_count,
                                              ctypes.byref(bt), _ptr(kv_lens), max_kv_len, w, _ptr(k_new), _ptr(v_new),
                                              _ptr(q), softmax_scale, _ptr(out), out_dtype, _ptr(lse), _ptr(workspace),
                                              workspace.numel() * workspace.element_size(), _ptr(status_flags), _stream()),
           "q4kv_decode_attention_layers")
