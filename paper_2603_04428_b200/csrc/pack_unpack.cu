// q4kv_pack / q4kv_unpack: the contiguous per-agent layout that is persisted and restored
// (Appendix A schema, groups along head_dim), gathered from / scattered into pool blocks
// through one block-table row.
//
// One CTA handles one (layer, logical block, KV head).  K words only change position
// inside their 32-token chunk; scale/bias pairs are split into two tensors; V codes are transposed
// between the pool's token-packed words and the persisted head-dim-packed words through a
// shared-memory tile of one byte per code, 32 tokens at a time.
#include "q4kv_layout.cuh"

namespace q4kv {

namespace {

constexpr int kThreads = 256;

struct PersistedOffsets { uint64_t kc, ks, kb, vc, vs, vb; };

__device__ inline PersistedOffsets persisted_offsets(const Layout& y) {
  PersistedOffsets o;
  const uint64_t T = kBlockTokens, H = y.Hkv;
  o.kc = 0;
  o.ks = o.kc + H * T * (y.D / 2);
  o.kb = o.ks + H * T * 2 * y.G;
  o.vc = o.kb + H * T * 2 * y.G;
  o.vs = o.vc + H * T * (y.Dv / 2);
  o.vb = o.vs + H * T * 2 * y.Gv;
  return o;
}

// grid: (n_logical_blocks * Hkv, L); dynamic smem 32 * Dv bytes (V transposition tile)
template <bool kPack>
__global__ void __launch_bounds__(kThreads)
pack_unpack_kernel(Layout y, uint8_t* pool, int n_blocks, const int32_t* __restrict__ row, int n_tokens,
                   uint8_t* buf, int32_t* flags) {
  extern __shared__ uint8_t tile[];   // [32 tokens][Dv] codes
  const int lb = blockIdx.x / y.Hkv, hk = blockIdx.x % y.Hkv, layer = blockIdx.y;
  const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;
  const int phys = row[lb];
  if (phys < 0 || phys >= n_blocks) {
    if (threadIdx.x == 0) raise_flag(flags, Q4KV_FLAG_BAD_BLOCK);
    if (!kPack) return;
  }
  const bool bad = phys < 0 || phys >= n_blocks;
  const int valid = min(kBlockTokens, n_tokens - lb * kBlockTokens);   // slots >= valid are zero bytes
  uint8_t* hb = bad ? nullptr : head_block(pool, y, layer, phys, hk);
  uint8_t* pb = buf + ((uint64_t)layer * nblk + lb) * persisted_block_bytes(y);
  const PersistedOffsets po = persisted_offsets(y);
  const int kw = y.D / 8, vw = y.Dv / 8;

  // K codes: word permutation inside each chunk
  {
    uint32_t* pk = reinterpret_cast<uint32_t*>(pb + po.kc) + (size_t)hk * kBlockTokens * kw;
    for (int i = threadIdx.x; i < kBlockTokens * kw; i += kThreads) {
      const int slot = i / kw, w = i % kw;
      uint32_t* dk = bad ? nullptr : reinterpret_cast<uint32_t*>(hb + (size_t)(slot >> 5) * y.chunk_bytes + y.off_kc) +
                                         k_word_offset(slot & 31, w, y.G);
      if (kPack) pk[i] = (slot < valid && !bad) ? *dk : 0u;
      else *dk = pk[i];
    }
  }
  // K and V scale / bias
  for (int which = 0; which < (y.alias ? 1 : 2); ++which) {
    const int G = which ? y.Gv : y.G;
    __half* ps = reinterpret_cast<__half*>(pb + (which ? po.vs : po.ks)) + (size_t)hk * kBlockTokens * G;
    __half* pbias = reinterpret_cast<__half*>(pb + (which ? po.vb : po.kb)) + (size_t)hk * kBlockTokens * G;
    for (int i = threadIdx.x; i < kBlockTokens * G; i += kThreads) {
      const int slot = i / G, gi = i % G;
      __half2* dsb = bad ? nullptr : reinterpret_cast<__half2*>(hb + (size_t)(slot >> 5) * y.chunk_bytes +
                                                                  (which ? y.off_vsb : y.off_ksb)) +
                                         sb_offset(slot & 31, gi, G);
      if (kPack) {
        __half2 v = __halves2half2(__ushort_as_half((unsigned short)0), __ushort_as_half((unsigned short)0));
        if (slot < valid && !bad) v = *dsb;
        ps[i] = __low2half(v);
        pbias[i] = __high2half(v);
      } else {
        *dsb = __halves2half2(ps[i], pbias[i]);
      }
    }
  }
  if (y.alias) return;
  // V codes: transpose 32 tokens at a time
  uint32_t* pv = reinterpret_cast<uint32_t*>(pb + po.vc) + (size_t)hk * kBlockTokens * vw;
  const int words = 4 * y.Dv;   // words of one 32-token chunk in either layout (32*Dv/8)
  for (int c = 0; c < 8; ++c) {
    uint32_t* dv = bad ? nullptr : reinterpret_cast<uint32_t*>(hb + (size_t)c * y.chunk_bytes + y.off_vc);
    if (kPack) {
      // pool word (element d, token octet o) -> tile[8o+k][d]
      for (int i = threadIdx.x; i < words; i += kThreads) {
        const int d = i >> 2, o = i & 3;
        const uint32_t w = bad ? 0u : dv[v_word_offset(o, d)];
#pragma unroll
        for (int k = 0; k < 8; ++k) tile[(8 * o + k) * y.Dv + d] = (w >> (4 * k)) & 15u;
      }
      __syncthreads();
      for (int i = threadIdx.x; i < words; i += kThreads) {
        const int tok = i / vw, w = i % vw;
        uint32_t o = 0;
        if (32 * c + tok < valid) {
#pragma unroll
          for (int k = 0; k < 8; ++k) o |= (uint32_t)tile[tok * y.Dv + 8 * w + k] << (4 * k);
        }
        pv[(size_t)(32 * c + tok) * vw + w] = o;
      }
      __syncthreads();
    } else {
      for (int i = threadIdx.x; i < words; i += kThreads) {
        const int tok = i / vw, w = i % vw;
        const uint32_t o = pv[(size_t)(32 * c + tok) * vw + w];
#pragma unroll
        for (int k = 0; k < 8; ++k) tile[tok * y.Dv + 8 * w + k] = (o >> (4 * k)) & 15u;
      }
      __syncthreads();
      for (int i = threadIdx.x; i < words; i += kThreads) {
        const int d = i >> 2, o = i & 3;
        uint32_t w = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) w |= (uint32_t)tile[(8 * o + k) * y.Dv + d] << (4 * k);
        dv[v_word_offset(o, d)] = w;
      }
      __syncthreads();
    }
  }
}

}  // namespace

cudaError_t launch_pack(const Layout& y, const void* pool, int n_blocks, const int32_t* row, int n_tokens,
                        void* dst, int32_t* flags, cudaStream_t st) {
  if (n_tokens <= 0) return cudaSuccess;
  const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;
  dim3 grid(nblk * y.Hkv, y.L);
  pack_unpack_kernel<true><<<grid, kThreads, y.alias ? 0 : 32 * y.Dv, st>>>(
      y, (uint8_t*)pool, n_blocks, row, n_tokens, (uint8_t*)dst, flags);
  return cudaGetLastError();
}

cudaError_t launch_unpack(const Layout& y, const void* src, int n_tokens, void* pool, int n_blocks,
                          const int32_t* row, int32_t* flags, cudaStream_t st) {
  if (n_tokens <= 0) return cudaSuccess;
  const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;
  dim3 grid(nblk * y.Hkv, y.L);
  pack_unpack_kernel<false><<<grid, kThreads, y.alias ? 0 : 32 * y.Dv, st>>>(
      y, (uint8_t*)pool, n_blocks, row, n_tokens, (uint8_t*)src, flags);
  return cudaGetLastError();
}

}  // namespace q4kv
