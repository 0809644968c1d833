// q4kv_pack / q4kv_unpack: the contiguous per-agent layout that is persisted and restored
// (Appendix A schema, groups along head_dim), gathered from / scattered into pool blocks
// through one block-table row.
//
// One CTA handles one (layer, logical block, KV head), one warp per 32-token chunk.  K words only
// change position inside their chunk; scale/bias pairs are split into two tensors; V codes are
// transposed between the pool's token-packed words and the persisted head-dim-packed words as
// 8x8 nibble blocks in registers.
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

// Transpose an 8x8 matrix of nibbles held as eight words (row r = a[r], column c in bits [4c, 4c+4)).
__device__ inline void transpose_nibbles_8x8(uint32_t (&a)[8]) {
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const uint32_t t = ((a[r] >> 16) ^ a[r + 4]) & 0x0000FFFFu;
    a[r + 4] ^= t; a[r] ^= t << 16;
  }
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    if (r & 2) continue;
    const uint32_t t = ((a[r] >> 8) ^ a[r + 2]) & 0x00FF00FFu;
    a[r + 2] ^= t; a[r] ^= t << 8;
  }
#pragma unroll
  for (int r = 0; r < 8; r += 2) {
    const uint32_t t = ((a[r] >> 4) ^ a[r + 1]) & 0x0F0F0F0Fu;
    a[r + 1] ^= t; a[r] ^= t << 4;
  }
}

// Where the head-dim-packed side of the exchange lives.  mode 0: the persisted per-agent buffer (whole blocks, layer
// outermost, starting at layer0).  mode 1: a dense left-padded batch of one layer (the paper's merged cache, Section
// 3.4): tensors K_codes [A][Hkv][T][d_qk/8], K_scales, K_biases [A][Hkv][T][d_qk/64], V likewise, one after the other;
// agent a's tokens occupy rows T - len_a .. T - 1.
struct ExchangeView {
  int mode, layer0, T, max_blocks, n_agents;
  const int32_t* lens;
};

// grid: (n_logical_blocks * Hkv, L) in mode 0, (n_logical_blocks * Hkv, A) in mode 1; 8 warps, warp c handles 32-token
// chunk c of the head-block through its own shared-memory copy of the chunk (dynamic smem: 8 * chunk_bytes).  Every
// global access is a full 16- or 32-byte piece of a contiguous run: the pool chunk is one contiguous range, and each
// head-dim-packed tensor's part of a chunk is too.
template <bool kPack, bool kDense>
__global__ void __launch_bounds__(kThreads)
pack_unpack_kernel(Layout y, uint8_t* pool, int n_blocks, const int32_t* __restrict__ row, int n_tokens,
                   uint8_t* buf, int32_t* flags, ExchangeView xv) {
  extern __shared__ __align__(16) uint8_t stage_all[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int lb = blockIdx.x / y.Hkv, hk = blockIdx.x % y.Hkv;
  const int kw = y.D / 8, vw = y.Dv / 8;
  int layer;
  uint8_t *b_kc, *b_ks, *b_kb, *b_vc, *b_vs, *b_vb;      // tensor bases; row index of this head-block's slot 0 below
  uint64_t row0;
  if (!kDense) {
    layer = xv.layer0 + blockIdx.y;                      // buf starts at layer0
    const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;
    uint8_t* pb = buf + ((uint64_t)blockIdx.y * nblk + lb) * persisted_block_bytes(y);
    const PersistedOffsets po = persisted_offsets(y);
    b_kc = pb + po.kc; b_ks = pb + po.ks; b_kb = pb + po.kb; b_vc = pb + po.vc; b_vs = pb + po.vs; b_vb = pb + po.vb;
    row0 = (uint64_t)hk * kBlockTokens;
  } else {
    layer = xv.layer0;
    const int a = blockIdx.y;
    row += (size_t)a * xv.max_blocks;
    n_tokens = xv.lens[a];
    if (n_tokens < 0 || n_tokens > xv.T || n_tokens > xv.max_blocks * kBlockTokens) {
      if (threadIdx.x == 0 && blockIdx.x == 0) raise_flag(flags, Q4KV_FLAG_BAD_LENGTH);
      return;
    }
    if (lb * kBlockTokens >= n_tokens) return;
    const uint64_t rows = (uint64_t)xv.n_agents * y.Hkv * xv.T;
    b_kc = buf; b_ks = b_kc + rows * kw * 4; b_kb = b_ks + rows * y.G * 2;
    b_vc = b_kb + rows * y.G * 2; b_vs = b_vc + rows * vw * 4; b_vb = b_vs + rows * y.Gv * 2;
    // may be "negative" for the first block of a short agent; only rows of existing tokens are ever touched
    row0 = ((uint64_t)a * y.Hkv + hk) * xv.T + (uint64_t)(xv.T - n_tokens) + (uint64_t)lb * kBlockTokens;
  }
  constexpr bool whole_blocks = !kDense;                // the persisted buffer holds whole blocks: rows past the end are zero bytes
  const int phys = row[lb];
  const bool bad = phys < 0 || phys >= n_blocks;
  if (bad) {
    if (threadIdx.x == 0) raise_flag(flags, Q4KV_FLAG_BAD_BLOCK);
    if (!kPack) return;
  }
  const int slot0 = warp * kChunkTokens;
  const int nv = max(0, min(kChunkTokens, n_tokens - lb * kBlockTokens - slot0));   // tokens of this chunk that exist
  const int nr = whole_blocks ? kChunkTokens : nv;       // rows of the chunk that exist on the head-dim-packed side
  if (nr == 0) return;
  uint8_t* chunk = bad ? nullptr : head_block(pool, y, layer, phys, hk) + (size_t)warp * y.chunk_bytes;
  uint8_t* st = stage_all + (size_t)warp * y.chunk_bytes;
  uint32_t* st_kc = reinterpret_cast<uint32_t*>(st + y.off_kc);
  __half2* st_ksb = reinterpret_cast<__half2*>(st + y.off_ksb);
  uint32_t* st_vc = reinterpret_cast<uint32_t*>(st + y.off_vc);
  __half2* st_vsb = reinterpret_cast<__half2*>(st + y.off_vsb);
  uint32_t* pk = reinterpret_cast<uint32_t*>(b_kc) + (row0 + slot0) * kw;
  uint32_t* pv = reinterpret_cast<uint32_t*>(b_vc) + (row0 + slot0) * vw;
  const __half hzero = __ushort_as_half((unsigned short)0);
  const int n16 = y.chunk_bytes / 16;

  if (kPack) {
    for (int u = lane; u < n16; u += 32)
      reinterpret_cast<uint4*>(st)[u] = (bad || nv == 0) ? make_uint4(0u, 0u, 0u, 0u) : reinterpret_cast<const uint4*>(chunk)[u];
    __syncwarp();
    // K codes: one 16-byte piece of a head-dim-packed row per lane and step
    for (int q = lane; q < nr * kw / 4; q += 32) {
      const int tau = q / (kw / 4), x0 = (q % (kw / 4)) * 4;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tau < nv) {
        v.x = st_kc[k_word_offset(tau, x0, y.G)]; v.y = st_kc[k_word_offset(tau, x0 + 1, y.G)];
        v.z = st_kc[k_word_offset(tau, x0 + 2, y.G)]; v.w = st_kc[k_word_offset(tau, x0 + 3, y.G)];
      }
      reinterpret_cast<uint4*>(pk)[q] = v;
    }
  } else {
    if (!whole_blocks && nv < kChunkTokens) {
      // a partly filled chunk of the pool keeps its other slots: start from its present bytes
      for (int u = lane; u < n16; u += 32) reinterpret_cast<uint4*>(st)[u] = reinterpret_cast<const uint4*>(chunk)[u];
      __syncwarp();
    }
    for (int q = lane; q < nr * kw / 4; q += 32) {
      const int tau = q / (kw / 4), x0 = (q % (kw / 4)) * 4;
      const uint4 v = reinterpret_cast<const uint4*>(pk)[q];
      st_kc[k_word_offset(tau, x0, y.G)] = v.x; st_kc[k_word_offset(tau, x0 + 1, y.G)] = v.y;
      st_kc[k_word_offset(tau, x0 + 2, y.G)] = v.z; st_kc[k_word_offset(tau, x0 + 3, y.G)] = v.w;
    }
  }
  // scales and biases: half2 (scale, bias) per token and group in the pool, two tensors on the other side
  for (int which = 0; which < (y.alias ? 1 : 2); ++which) {
    const int G = which ? y.Gv : y.G;
    __half* ps = reinterpret_cast<__half*>(which ? b_vs : b_ks) + (row0 + slot0) * G;
    __half* pbias = reinterpret_cast<__half*>(which ? b_vb : b_kb) + (row0 + slot0) * G;
    __half2* stsb = which ? st_vsb : st_ksb;
    for (int i = lane; i < nr * G; i += 32) {
      const int tau = i / G, gi = i % G;
      if (kPack) {
        const __half2 v = tau < nv ? stsb[sb_offset(tau, gi, G)] : __halves2half2(hzero, hzero);
        ps[i] = __low2half(v);
        pbias[i] = __high2half(v);
      } else {
        stsb[sb_offset(tau, gi, G)] = __halves2half2(ps[i], pbias[i]);
      }
    }
  }
  // V codes: 8x8 nibble blocks (8 tokens x 8 head-dim elements) transposed in registers
  if (!y.alias) {
    const int o = lane >> 3;                      // token octet of the chunk
    for (int w = lane & 7; w < vw; w += 8) {      // head-dim-packed word index inside a row
      uint32_t a[8];
      if (kPack) {
#pragma unroll
        for (int j = 0; j < 8; ++j) a[j] = st_vc[v_word_offset(o, 8 * w + j)];
        transpose_nibbles_8x8(a);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (8 * o + k < nr) pv[(size_t)(8 * o + k) * vw + w] = (8 * o + k < nv) ? a[k] : 0u;
      } else {
        if (8 * o >= nr) continue;
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = (8 * o + k < nr) ? pv[(size_t)(8 * o + k) * vw + w] : 0u;
        transpose_nibbles_8x8(a);
        // positions of the octet that do not exist on the other side keep the pool's nibbles
        const int have = min(8, nr - 8 * o);
        const uint32_t m = have >= 8 ? 0xFFFFFFFFu : ((1u << (4 * have)) - 1u);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t* at = &st_vc[v_word_offset(o, 8 * w + j)];
          *at = m == 0xFFFFFFFFu ? a[j] : ((*at & ~m) | (a[j] & m));
        }
      }
    }
  }
  if (!kPack) {
    __syncwarp();
    for (int u = lane; u < n16; u += 32) reinterpret_cast<uint4*>(chunk)[u] = reinterpret_cast<const uint4*>(st)[u];
  }
}

}  // namespace

namespace {
template <bool kPack, bool kDense>
cudaError_t launch_pu(const Layout& y, uint8_t* pool, int n_blocks, const int32_t* row, int n_tokens, uint8_t* buf,
                      int32_t* flags, cudaStream_t st, const ExchangeView& xv, int grid_y) {
  static bool configured[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(pack_unpack_kernel<kPack, kDense>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;   // mode 1: n_tokens is T, the dense row count
  dim3 grid(nblk * y.Hkv, grid_y);
  pack_unpack_kernel<kPack, kDense><<<grid, kThreads, (size_t)kChunksPerBlock * y.chunk_bytes, st>>>(y, pool, n_blocks, row, n_tokens,
                                                                                              buf, flags, xv);
  return cudaGetLastError();
}
ExchangeView persisted_view(int layer0) {
  ExchangeView xv;
  xv.mode = 0; xv.layer0 = layer0; xv.T = 0; xv.max_blocks = 0; xv.n_agents = 0; xv.lens = nullptr;
  return xv;
}
}  // namespace

cudaError_t launch_pack(const Layout& y, const void* pool, int n_blocks, const int32_t* row, int n_tokens,
                        void* dst, int32_t* flags, cudaStream_t st) {
  if (n_tokens <= 0) return cudaSuccess;
  return launch_pu<true, false>(y, (uint8_t*)pool, n_blocks, row, n_tokens, (uint8_t*)dst, flags, st, persisted_view(0), y.L);
}

cudaError_t launch_unpack(const Layout& y, const void* src, int n_tokens, void* pool, int n_blocks,
                          const int32_t* row, int32_t* flags, cudaStream_t st) {
  if (n_tokens <= 0) return cudaSuccess;
  return launch_pu<false, false>(y, (uint8_t*)pool, n_blocks, row, n_tokens, (uint8_t*)src, flags, st, persisted_view(0), y.L);
}

// layers [layer0, layer0 + layer_count) only; src points at the persisted bytes of layer0
cudaError_t launch_unpack_layers(const Layout& y, const void* src, int n_tokens, void* pool, int n_blocks,
                                 const int32_t* row, int32_t* flags, cudaStream_t st, int layer0, int layer_count) {
  if (n_tokens <= 0 || layer_count <= 0) return cudaSuccess;
  return launch_pu<false, false>(y, (uint8_t*)pool, n_blocks, row, n_tokens, (uint8_t*)src, flags, st, persisted_view(layer0), layer_count);
}

// the dense left-padded batch of one layer <-> the pool (to_pool: the paper's merge; else extract, into a zeroed buffer)
cudaError_t launch_dense_exchange(const Layout& y, void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                  const int32_t* kv_lens, int T, void* dense, bool to_pool, int32_t* flags, cudaStream_t st) {
  if (b.n_agents <= 0 || T <= 0) return cudaSuccess;
  ExchangeView xv;
  xv.mode = 1; xv.layer0 = layer; xv.T = T; xv.max_blocks = b.max_blocks; xv.n_agents = b.n_agents; xv.lens = kv_lens;
  if (to_pool) return launch_pu<false, true>(y, (uint8_t*)pool, n_blocks, b.block_tables, T, (uint8_t*)dense, flags, st, xv, b.n_agents);
  return launch_pu<true, true>(y, (uint8_t*)pool, n_blocks, b.block_tables, T, (uint8_t*)dense, flags, st, xv, b.n_agents);
}

}  // namespace q4kv
