"""Device-side cache holder used by the tests, the smoke check and the benchmark.

It only allocates torch CUDA tensors (pool, block tables, lengths, workspace,
status word) and forwards to the C-ABI binding; no step of the method runs
here.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


class DeviceCache:
    def __init__(self, n_layers, n_q_heads, n_kv_heads, d_qk, d_v, v_aliases_k, n_blocks, block_tables: np.ndarray,
                 fill_byte: int | None = 0xFF, exact_products: bool = False, sb_dtype: int = 0):
        self.spec = B.Spec.make(n_layers, n_q_heads, n_kv_heads, d_qk, d_v, v_aliases_k, exact_products, sb_dtype)
        self.n_blocks = int(n_blocks)
        nbytes = B.q4kv_pool_bytes(self.spec, self.n_blocks)
        assert nbytes > 0, "unsupported spec"
        self.pool = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        if fill_byte is not None:
            self.pool.fill_(fill_byte)       # 0xFF: stale slots hold NaN scale bits on purpose
        self.tables = dev(block_tables.astype(np.int32))
        self.bt = B.batch(self.tables)
        self.flags = torch.zeros(1, dtype=torch.int32, device="cuda")
        self._ws = None

    # ---- helpers -------------------------------------------------------------------------------
    def sub_batch(self, a0, a1):
        t = self.tables[a0:a1].contiguous()
        return t, B.batch(t)

    def workspace(self, n_agents, max_kv_len, total_q=0):
        need = B.q4kv_workspace_bytes(self.spec, n_agents, max_kv_len, total_q)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.zeros(need, dtype=torch.uint8, device="cuda")   # arrival counters start at zero
        return self._ws

    def read_flags(self) -> int:
        return int(self.flags.item())

    # ---- the five operations -------------------------------------------------------------------
    def append(self, layer, pos, new_offs, k_bits, v_bits, bt=None):
        """k_bits/v_bits: numpy uint16 [total_new][Hkv][d] or CUDA bf16 tensors."""
        k = bf16_dev(k_bits) if isinstance(k_bits, np.ndarray) else k_bits
        v = None
        if v_bits is not None:
            v = bf16_dev(v_bits) if isinstance(v_bits, np.ndarray) else v_bits
        pos_d = dev(np.asarray(pos, dtype=np.int32)) if not torch.is_tensor(pos) else pos
        offs_d = dev(np.asarray(new_offs, dtype=np.int32)) if not torch.is_tensor(new_offs) else new_offs
        total_new = int(k.shape[0])
        B.q4kv_quantize_append(self.spec, self.pool, self.n_blocks, layer, bt or self.bt, pos_d, offs_d, total_new,
                               k, v, self.flags)

    def decode(self, layer, kv_lens, window, q_bits, scale, out_dtype=B.OUT_F32, want_lse=True, bt=None,
               max_kv_len=0):
        q = bf16_dev(q_bits) if isinstance(q_bits, np.ndarray) else q_bits
        A = q.shape[0]
        lens_d = dev(np.asarray(kv_lens, dtype=np.int32)) if not torch.is_tensor(kv_lens) else kv_lens
        out = torch.empty((A, self.spec.n_q_heads, self.spec.d_v), device="cuda",
                          dtype=torch.float32 if out_dtype == B.OUT_F32 else torch.bfloat16)
        lse = torch.empty((A, self.spec.n_q_heads), dtype=torch.float32, device="cuda") if want_lse else None
        b = bt or self.bt
        cap = b.max_blocks * 256
        ws = self.workspace(A, max_kv_len or cap)
        B.q4kv_decode_attention(self.spec, self.pool, self.n_blocks, layer, b, lens_d, max_kv_len, window, q,
                                float(scale), out, out_dtype, lse, ws, self.flags)
        return out, lse

    def append_decode(self, layer, kv_lens, window, k_bits, v_bits, q_bits, scale, out_dtype=B.OUT_F32, bt=None):
        """One new token per agent appended at position kv_len - 1 and attended, in one launch."""
        q = bf16_dev(q_bits) if isinstance(q_bits, np.ndarray) else q_bits
        k = bf16_dev(k_bits) if isinstance(k_bits, np.ndarray) else k_bits
        v = bf16_dev(v_bits) if isinstance(v_bits, np.ndarray) else v_bits
        A = q.shape[0]
        lens_d = dev(np.asarray(kv_lens, dtype=np.int32)) if not torch.is_tensor(kv_lens) else kv_lens
        out = torch.empty((A, self.spec.n_q_heads, self.spec.d_v), device="cuda",
                          dtype=torch.float32 if out_dtype == B.OUT_F32 else torch.bfloat16)
        lse = torch.empty((A, self.spec.n_q_heads), dtype=torch.float32, device="cuda")
        b = bt or self.bt
        ws = self.workspace(A, b.max_blocks * 256)
        B.q4kv_append_decode_attention(self.spec, self.pool, self.n_blocks, layer, b, lens_d, 0, window, k, v, q,
                                       float(scale), out, out_dtype, lse, ws, self.flags)
        return out, lse

    def prefill(self, layer, kv_lens, q_offs, window, q_bits, scale, out_dtype=B.OUT_F32, want_lse=True, bt=None,
                max_kv_len=0):
        q = bf16_dev(q_bits) if isinstance(q_bits, np.ndarray) else q_bits
        total_q = int(q.shape[0])
        q_offs = np.asarray(q_offs, dtype=np.int32)
        max_q_len = int(np.max(np.diff(q_offs))) if len(q_offs) > 1 else 0
        lens_d = dev(np.asarray(kv_lens, dtype=np.int32))
        offs_d = dev(q_offs)
        out = torch.empty((total_q, self.spec.n_q_heads, self.spec.d_v), device="cuda",
                          dtype=torch.float32 if out_dtype == B.OUT_F32 else torch.bfloat16)
        lse = torch.empty((total_q, self.spec.n_q_heads), dtype=torch.float32, device="cuda") if want_lse else None
        b = bt or self.bt
        cap = b.max_blocks * 256
        ws = self.workspace(len(kv_lens), max_kv_len or cap, total_q)
        B.q4kv_prefill_attention(self.spec, self.pool, self.n_blocks, layer, b, lens_d, offs_d, total_q, max_q_len,
                                 max_kv_len, window, q, float(scale), out, out_dtype, lse, ws, self.flags)
        return out, lse

    def pack(self, agent, n_tokens) -> torch.Tensor:
        dst = torch.empty(B.q4kv_packed_bytes(self.spec, n_tokens), dtype=torch.uint8, device="cuda")
        B.q4kv_pack(self.spec, self.pool, self.n_blocks, self.tables[agent], n_tokens, dst, self.flags)
        return dst

    def unpack(self, agent, n_tokens, buf):
        src = dev(buf) if isinstance(buf, np.ndarray) else buf
        B.q4kv_unpack(self.spec, src, n_tokens, self.pool, self.n_blocks, self.tables[agent], self.flags)

    # ---- persisted container and warm restore ----------------------------------------------------
    def save(self, agent, n_tokens) -> torch.Tensor:
        """The agent's file image (header + packed bytes) in pinned host memory."""
        hb = B.q4kv_container_header_bytes(self.spec, n_tokens)
        pb = B.q4kv_packed_bytes(self.spec, n_tokens)
        stage = torch.empty(pb, dtype=torch.uint8, device="cuda")
        image = torch.empty(hb + pb, dtype=torch.uint8).pin_memory()
        B.q4kv_save(self.spec, self.pool, self.n_blocks, self.tables[agent], n_tokens, stage, image, self.flags)
        torch.cuda.current_stream().synchronize()
        return image

    def restore(self, agent, image: torch.Tensor, staging_layers: int = 0):
        """Scatter a file image (pinned host uint8 tensor) into the agent's blocks; returns the token count."""
        spec, n_tokens, off = B.q4kv_container_read_header(bytes(image[:min(image.numel(), 1 << 22)].numpy()))
        same = all(getattr(spec, f) == getattr(self.spec, f) for f in (
            "n_layers", "n_q_heads", "n_kv_heads", "d_qk", "d_v", "v_aliases_k", "group", "block_tokens", "sb_dtype"))
        if not same:
            raise B.Q4KVError(-1, "restore: the image was written for another cache spec")
        pb = B.q4kv_packed_bytes(self.spec, n_tokens)
        packed = image[off:off + pb]
        if packed.data_ptr() % 16:
            packed = packed.clone().pin_memory()
        layer_bytes = pb // self.spec.n_layers
        n_stage = staging_layers or min(self.spec.n_layers, 8)
        stage = torch.empty(n_stage * layer_bytes, dtype=torch.uint8, device="cuda")
        copy_stream = torch.cuda.Stream()
        cur = torch.cuda.current_stream()
        copy_stream.wait_stream(cur)
        B.q4kv_restore(self.spec, packed, n_tokens, self.pool, self.n_blocks, self.tables[agent], stage, self.flags,
                       copy_stream=copy_stream, unpack_stream=cur)
        cur.synchronize()
        copy_stream.synchronize()
        return n_tokens

