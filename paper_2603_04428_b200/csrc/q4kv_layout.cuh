// Device-side layout of the Q4 block pool and small shared helpers.
//
// The pool's byte layout is private to this library (include/q4kv.h): it is arranged so that
// (a) any run of 32-token chunks of one KV head is ONE contiguous byte range (one bulk copy
// into shared memory), and (b) inside a chunk every warp-wide 16-byte shared-memory load is a
// contiguous 512-byte line whose words land directly in the register slots of the
// m16n8k16 tensor-core fragments (no shuffles, no bank conflicts).  The persisted layout of
// Appendix A is produced/consumed only by the pack/unpack kernels.
//
// pool = [n_layers][n_blocks][n_kv_heads] "head-blocks"; one head-block = 8 chunks; one chunk
// holds 32 consecutive tokens of one KV head of one layer:
//
//   chunk = [ Kc | Ksb | Vc | Vsb ]                       (Vc, Vsb absent when V aliases K)
//
// Names: chunk token tau in 0..31; fragment coordinates g = lane/4 (0..7), tid = lane%4.
//
//   Kc  : D/8 uint32 per token.  Logical word w holds head-dim elements 8w..8w+7 (element k in
//         bits [4k,4k+4)), w = 8*gi + 4*i2 + tid (gi = 64-element group, i2 in {0,1}).  Token
//         tau = 4*g + i belongs to key tile i (the 8 tokens 4g+i, g = 0..7).  A lane's 2G words
//         p = 2*gi + i2 are cut in pieces of 4 words (16 bytes):
//             word offset = i*64G + (p/4)*128 + (g*4 + tid)*pw + p%4,   pw = min(4, 2G - 4*(p/4))
//         so one 16-byte load per lane (g, tid) fetches a whole piece of tile i for the warp.
//   Ksb : G half2 (x = scale, y = bias) per token; token tau = 8*tid + 4*e + i sits at
//             half2 offset = ((i*4 + tid)*2 + e)*G + gi
//         (the two tokens a lane owns in the score fragment of tile i are adjacent).
//   Vc  : token-packed ("V transposed"): one uint32 holds the codes of ONE head-dim element d
//         for the 8 tokens 8*tid..8*tid+7 (token 8*tid+k in bits [4k,4k+4)).  With d = 16*mt + r,
//             word offset = (((mt/2)*8 + r%8)*4 + tid)*4 + (mt%2)*2 + r/8
//         so one 16-byte load per lane fetches rows g and g+8 of two 16-row value tiles.
//   Vsb : Gv half2 per token, arranged like Ksb; groups are still along head_dim.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/q4kv.h"

namespace q4kv {

constexpr int kBlockTokens = 256;
constexpr int kGroup = 64;
constexpr int kChunkTokens = 32;
constexpr int kChunksPerBlock = kBlockTokens / kChunkTokens;
// Head of every decode workspace: arrival counters of the split merge, one per (agent, KV head) pair, at zero
// between calls.  Its size does not depend on the call, so calls of any shape can share one workspace.
constexpr size_t kWorkspaceHeaderBytes = Q4KV_WORKSPACE_HEADER_BYTES;
constexpr int kMaxTicketPairs = (int)(kWorkspaceHeaderBytes / sizeof(int32_t));

struct Layout {
  int L, Hq, Hkv, D, Dv, G, Gv, alias, n_rep;
  int sb_bf16;            // scales and biases are bfloat16 (else binary16)
  // byte offsets inside a chunk
  uint32_t off_kc, off_ksb, off_vc, off_vsb, chunk_bytes, head_block_bytes;
  uint64_t block_bytes;   // all KV heads
  uint64_t layer_bytes;   // n_blocks * block_bytes
};

__host__ __device__ inline Layout make_layout(const q4kv_spec& s, int n_blocks) {
  Layout y;
  y.L = s.n_layers; y.Hq = s.n_q_heads; y.Hkv = s.n_kv_heads; y.D = s.d_qk; y.Dv = s.d_v;
  y.G = s.d_qk / kGroup; y.Gv = s.d_v / kGroup; y.alias = s.v_aliases_k ? 1 : 0;
  y.n_rep = s.n_q_heads / s.n_kv_heads;
  y.sb_bf16 = s.sb_dtype == 1 ? 1 : 0;
  y.off_kc = 0;
  y.off_ksb = kChunkTokens * (y.D / 2);
  y.off_vc = y.off_ksb + kChunkTokens * 4 * y.G;
  y.off_vsb = y.off_vc + (y.alias ? 0 : kChunkTokens * (y.Dv / 2));
  y.chunk_bytes = y.off_vsb + (y.alias ? 0 : kChunkTokens * 4 * y.Gv);
  y.head_block_bytes = kChunksPerBlock * y.chunk_bytes;
  y.block_bytes = (uint64_t)y.Hkv * y.head_block_bytes;
  y.layer_bytes = (uint64_t)n_blocks * y.block_bytes;
  return y;
}

// persisted (Appendix A) bytes of one block, all heads
__host__ __device__ inline uint64_t persisted_block_bytes(const Layout& y) {
  return (uint64_t)kBlockTokens * y.Hkv * (y.D / 2 + 4 * y.G + (y.alias ? 0 : (y.Dv / 2 + 4 * y.Gv)));
}

// uint32 offset inside a chunk's Kc of logical word w (elements 8w..8w+7) of chunk token tau
__host__ __device__ inline int k_word_offset(int tau, int w, int G) {
  const int i = tau & 3, g = tau >> 2;
  const int gi = w >> 3, i2 = (w >> 2) & 1, tid = w & 3;
  const int p = 2 * gi + i2, j = p >> 2;
  const int rest = 2 * G - 4 * j, pw = rest < 4 ? rest : 4;
  return i * 64 * G + j * 128 + (g * 4 + tid) * pw + (p & 3);
}
// half2 offset inside a chunk's Ksb / Vsb of (chunk token tau, group gi)
__host__ __device__ inline int sb_offset(int tau, int gi, int G) {
  const int i = tau & 3, e = (tau >> 2) & 1, tid = tau >> 3;
  return ((i * 4 + tid) * 2 + e) * G + gi;
}
// uint32 offset inside a chunk's Vc of the word holding element d for token octet o (tokens 8o..8o+7)
__host__ __device__ inline int v_word_offset(int o, int d) {
  const int mt = d >> 4, r = d & 15;
  return ((((mt >> 1) * 8 + (r & 7)) * 4 + o) * 4) + (mt & 1) * 2 + (r >> 3);
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
cudaError_t launch_unpack_layers(const Layout& y, const void* src, int n_tokens, void* pool, int n_blocks,
                                 const int32_t* row, int32_t* flags, cudaStream_t st, int layer0, int layer_count);
cudaError_t launch_dense_exchange(const Layout& y, void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                  const int32_t* kv_lens, int T, void* dense, bool to_pool, int32_t* flags, cudaStream_t st);
cudaError_t launch_attention_generic(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                     const int32_t* kv_lens, const int32_t* q_offs, int total_q, int max_q_len,
                                     int max_kv_len, int window, const void* q, float scale, void* out,
                                     int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st);

// tensor-core decode path (GQA shapes with d_qk = d_v in {128, 256}, at most 4 query heads per KV head)
bool decode_mma_supported(const Layout& y);
bool decode_mma_fits(const Layout& y, int n_agents, int max_blocks, int layer_count = 1);
int sm_count();   // SMs of the current device (148 when no device can be asked)
size_t decode_mma_workspace_bytes(const Layout& y, int n_agents, int layer_count = 1);
cudaError_t launch_decode_mma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                              const int32_t* kv_lens, int max_kv_len, const int32_t* windows, int layer_count,
                              const void* q, float scale, void* out, int out_dtype, float* lse, void* ws, int32_t* flags,
                              cudaStream_t st, const void* k_new = nullptr, const void* v_new = nullptr);

// tensor-core prefill path (d_qk = d_v = 128, at most 4 query heads per KV head)
bool prefill_mma_supported(const Layout& y);
cudaError_t launch_prefill_mma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                               const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window, const void* q,
                               float scale, void* out, int out_dtype, float* lse, int32_t* flags, cudaStream_t st);


// tcgen05 prefill path (d_qk = d_v = 128; 1, 2 or 4 query heads per KV head)
bool prefill_umma_supported(const Layout& y);
cudaError_t launch_prefill_umma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window, const void* q,
                                float scale, void* out, int out_dtype, float* lse, int32_t* flags, cudaStream_t st);

// tcgen05 prefill path for d_qk = d_v = 256 and for d_qk 192 / d_v 128 (1, 2 or 4 query heads per KV head): one 128-row
// tile per CTA, two score buffers
bool prefill_umma_1tile_supported(const Layout& y);
cudaError_t launch_prefill_umma_1tile(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                   const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window,
                                   const void* q, float scale, void* out, int out_dtype, float* lse, int32_t* flags,
                                   cudaStream_t st);

// Decode on the MLA-latent cache (d_qk 576, d_v 512 aliasing K, one KV head, at most 16 query heads): a key-split
// attention kernel -- on a binary16 tile of the dequantized keys, or, with on_codes, on the 4-bit codes themselves
// (exact products) -- followed by the combination of the records.
bool decode_mla_supported(const Layout& y);
size_t decode_mla_workspace_bytes(const Layout& y, int n_agents, int max_kv_len);
cudaError_t launch_decode_mla(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                              const int32_t* kv_lens, int max_kv_len, int window, const void* q, float scale, void* out,
                              int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st,
                              const void* k_new = nullptr,    // k_new: update-and-fetch (the pool is written)
                              bool on_codes = false);
// what the two attention kernels receive
struct MlaDecodeParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks;
  const int32_t* tables;
  const int32_t* kv_lens;
  int len_cap;
  int window;
  const uint16_t* q;          // bf16 [n_agents][Hq][576]
  const uint16_t* k_new;      // bf16 [n_agents][576]: the row at position kv_len - 1, quantized and stored by this launch; or null
  float scale_log2;
  int n_splits, blocks_per_split;
  float* records;             // [n_agents][n_splits][16][514]: acc[512] (unnormalised, relative to m), m, l
  int32_t* flags;
};
cudaError_t launch_mla_codes_kernel(const MlaDecodeParams& P, cudaStream_t st);   // grid (n_splits, n_agents)

}  // namespace q4kv
