// Device-side layout of the Q4 block pool and small shared helpers.
//
// The pool's byte layout is private to this library (include/q4kv.h): it is arranged so
// that the attention kernels' warp-level loads are contiguous 16-byte accesses and feed
// integer tensor-core fragments without shuffles.  The persisted layout of Appendix A is
// produced/consumed only by the pack/unpack kernels.
//
// pool = [n_layers][n_blocks][n_kv_heads] "head-blocks"; one head-block holds 256 tokens of
// one KV head of one layer:
//
//   Kc  : [256 tokens][D/8 words] uint32.  A logical word w of a row holds head-dim elements
//         8w..8w+7 (element k in bits [4k,4k+4)), w = 8*gi + 4*i2 + t with gi the 64-element
//         group, i2 in {0,1}, t in 0..3.  Physical position inside the row:
//             phys(w) = t*(2G) + 2*gi + i2          (G = D/64)
//         so the words one lane of a 4-lane quad needs (fixed t, all gi, i2) are contiguous.
//   Ksb : [256 tokens][G] half2 (x = scale, y = bias).
//   Vc  : [8 chunks of 32 tokens][Dv/32][8 g][4 t][4 j] uint32, token-packed ("V transposed"):
//         the word at (chunk c, J, g, t, j) belongs to head-dim element d = 32J + 8j + g and
//         holds tokens 32c + 8t + k, k = 0..7, in bits [4k,4k+4).   (absent when V aliases K)
//   Vsb : [256 tokens][Gv] half2 (scale, bias); groups are still along head_dim.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/q4kv.h"

namespace q4kv {

constexpr int kBlockTokens = 256;
constexpr int kGroup = 64;

struct Layout {
  int L, Hq, Hkv, D, Dv, G, Gv, alias, n_rep;
  // byte offsets inside a head-block
  uint32_t off_kc, off_ksb, off_vc, off_vsb, head_block_bytes;
  uint64_t block_bytes;   // all KV heads
  uint64_t layer_bytes;   // n_blocks * block_bytes (filled by make_layout with n_blocks)
};

__host__ __device__ inline Layout make_layout(const q4kv_spec& s, int n_blocks) {
  Layout y;
  y.L = s.n_layers; y.Hq = s.n_q_heads; y.Hkv = s.n_kv_heads; y.D = s.d_qk; y.Dv = s.d_v;
  y.G = s.d_qk / kGroup; y.Gv = s.d_v / kGroup; y.alias = s.v_aliases_k ? 1 : 0;
  y.n_rep = s.n_q_heads / s.n_kv_heads;
  y.off_kc = 0;
  y.off_ksb = kBlockTokens * (y.D / 2);
  y.off_vc = y.off_ksb + kBlockTokens * 4 * y.G;
  y.off_vsb = y.off_vc + (y.alias ? 0 : kBlockTokens * (y.Dv / 2));
  y.head_block_bytes = y.off_vsb + (y.alias ? 0 : kBlockTokens * 4 * y.Gv);
  y.block_bytes = (uint64_t)y.Hkv * y.head_block_bytes;
  y.layer_bytes = (uint64_t)n_blocks * y.block_bytes;
  return y;
}

// persisted (Appendix A) bytes of one block, all heads
__host__ __device__ inline uint64_t persisted_block_bytes(const Layout& y) {
  return (uint64_t)kBlockTokens * y.Hkv * (y.D / 2 + 4 * y.G + (y.alias ? 0 : (y.Dv / 2 + 4 * y.Gv)));
}

__host__ __device__ inline int k_phys_word(int w, int G) {
  const int gi = w >> 3, i2 = (w >> 2) & 1, t = w & 3;
  return t * (2 * G) + 2 * gi + i2;
}
__host__ __device__ inline int k_logical_word(int p, int G) {
  const int t = p / (2 * G), r = p % (2 * G);
  return 8 * (r >> 1) + 4 * (r & 1) + t;
}
// word index inside Vc of (token slot in block, head-dim element d)
__host__ __device__ inline int v_word_index(int slot, int d, int Dv) {
  const int c = slot >> 5, t = (slot >> 3) & 3;
  const int J = d >> 5, j = (d >> 3) & 3, g = d & 7;
  return (((c * (Dv >> 5) + J) * 8 + g) * 4 + t) * 4 + j;
}

__device__ inline const uint8_t* head_block(const void* pool, const Layout& y, int layer, int block, int kv_head) {
  return (const uint8_t*)pool + (uint64_t)layer * y.layer_bytes + (uint64_t)block * y.block_bytes +
         (uint64_t)kv_head * y.head_block_bytes;
}
__device__ inline uint8_t* head_block(void* pool, const Layout& y, int layer, int block, int kv_head) {
  return (uint8_t*)pool + (uint64_t)layer * y.layer_bytes + (uint64_t)block * y.block_bytes +
         (uint64_t)kv_head * y.head_block_bytes;
}

__device__ inline void raise_flag(int32_t* status_flags, int bit) {
  if (status_flags) atomicOr(status_flags, bit);
}

__device__ inline float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// host-side launch helpers (defined in the kernel translation units)
struct DecodePlan { int n_splits, split_tokens; };
DecodePlan plan_decode(const Layout& y, int n_agents, int max_kv_len, int window);

cudaError_t launch_quantize_append(const Layout& y, void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                   const int32_t* pos, const int32_t* new_offs, int total_new,
                                   const void* k_new, const void* v_new, int32_t* flags, cudaStream_t st);
cudaError_t launch_pack(const Layout& y, const void* pool, int n_blocks, const int32_t* row, int n_tokens,
                        void* dst, int32_t* flags, cudaStream_t st);
cudaError_t launch_unpack(const Layout& y, const void* src, int n_tokens, void* pool, int n_blocks,
                          const int32_t* row, int32_t* flags, cudaStream_t st);
cudaError_t launch_attention_generic(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                     const int32_t* kv_lens, const int32_t* q_offs, int total_q, int max_q_len,
                                     int max_kv_len, int window, const void* q, float scale, void* out,
                                     int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st);

}  // namespace q4kv
