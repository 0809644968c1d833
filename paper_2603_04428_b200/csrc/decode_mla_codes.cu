// q4kv_decode_attention for the MLA-latent cache, on the 4-bit codes (d_qk = 576 = 512 latent + 64 rope,
// d_v = 512, V aliases the first 512 dims of K, one shared KV head, up to 16 query heads): the route of
// calls that ask for exact products and of sharp softmax scales, for either scale / bias type
// (Section 3.4 "Batched Quantized Inference"; the MLA cache of Section 3.6).
//
// Every key serves all 16 heads and is both key and value, and both products run on the codes
// themselves (mma.sync m16n8k16 f16; a nibble masked in place in a 16-bit lane is the binary16
// subnormal c * 2^-24 or 16 c * 2^-24), so no dequantized tile is ever built and nothing of the cache
// is rounded:
//   * Work is split along the keys: CTA (split, agent) walks its share of the agent's keys 64 at a
//     time (two 32-token chunks = one bulk copy of 20736 bytes into a four-slot ring, issued by one
//     thread), leaves an (acc, m, l) record per head, and the record combination of the tile kernel's
//     file merges the records of an agent.
//   * Scores: warp W owns one key tile of the block (the 8 tokens 4g + i of one chunk): S[16 heads]
//     [8 keys] by 36 products whose B operand is the packed key word under a mask and whose A operand
//     is the query (binary16, each head scaled by a power of two; all 36 x 4 fragment registers stay
//     in registers for the whole launch).  Per 64-element group the integer dot product meets the
//     token's scale and the token's bias meets the per-group query sum, in float32: the scores are
//     exact up to float32 rounding, whatever the softmax scale.
//   * The warp also stores its key words again, regrouped so that the 16-byte rows of one group of 64
//     dims lie together: the value product reads them with ldmatrix.trans, which turns "four dims
//     of one token per 16-bit element" into "one 16-bit element of two tokens per register" -- after
//     the same masks, exactly the A operand of a product over tokens.  The bytes are moved, never
//     dequantized.
//   * Values: warp w owns the 64 dims of group w: O^T[64 dims][16 heads] += V^T (P s_w)^T.  The
//     probabilities travel through shared memory as float32 pairs in the fragment order of the B
//     operand (the lane that computed a pair is the lane that needs it, in every warp), are multiplied
//     by the tokens' scales of group w in float32 and enter the product as a two-term binary16 pair
//     (64 products per block), and meet the tokens' biases in float32.  The codes that sit four bits
//     up inside their 16-bit lane accumulate 16 times their value in accumulators of their own; the
//     factor is divided out when the record is written.
//   * Softmax with a lazily moved reference maximum per head, shared by the CTA: probabilities are
//     taken against the current reference; a block whose scores exceed it by more than 2^3 raises a
//     flag, and then (rarely: the first block, and when the maximum grows) the block's exact
//     per-head maximum becomes the reference, the accumulators are rescaled and the block's
//     probabilities are retaken.  One CTA-wide barrier per block otherwise.
// The raw blocks arrive on mbarriers with bounded waits (Q4KV_FLAG_INTERNAL when one runs out; the
// 256 threads then leave together).  Eight warps: the query fragments alone take 144 registers.
#include "q4kv_layout.cuh"
#include "quantize_core.cuh"
#include "tcgen05.cuh"

namespace q4kv {

namespace {

using namespace tc;   // mbarrier and bulk-copy wrappers

constexpr int kD = 576, kDv = 512, kHeads = 16, kG = kD / 64, kGv = kDv / 64;
constexpr int kComputeWarps = 8;
constexpr int kThreads = kComputeWarps * 32;            // 256
constexpr int kChunkBytes = 32 * (kD / 2 + 4 * kG);      // 10368: [Kc 9216 | Ksb 1152]
constexpr int kRawBytes = 2 * kChunkBytes;               // one 64-key block
constexpr int kRawSlots = 4;
constexpr int kRecStride = kDv + 2;                      // acc[512], m, l
constexpr float kLazy = 3.f;                             // probabilities stay below 2^3: p * scale fits binary16 for any binary16 scale
constexpr uint32_t kMaskLo = 0x000F000Fu, kMaskHi = 0x00F000F0u;

using MlaParams = MlaDecodeParams;

struct MlaSmem {
  alignas(128) uint8_t raw[kRawSlots][kRawBytes];
  // key words regrouped for the value product: [buffer][group 8][key tile 8][half row 2][token row 8][16 bytes]
  alignas(128) uint8_t vre[2][kGv * 8 * 2 * 8 * 16];
  // query A fragments [product 36][lane 32] = {a0, a1, a2, a3}; only read while the fragments are loaded into registers
  alignas(16) uint4 qfrag[kD / 16][32];
  float2 ptile[2][8][2][32];                             // [buffer][key tile][heads 0-7 | 8-15][lane] = p of the lane's two tokens
  uint32_t stab[2][kGv][8][4];                           // [buffer][group][key tile][tid] = the 16-bit scales of the two tokens
  uint32_t btab[2][kGv][8][4];                           // likewise the biases
  float kappa[kHeads];                                   // score in log2 units = integer dot product * scale * kappa[head] + ...
  float qsum[kHeads][kG];                                // scale_log2 * sum of the true q over each group
  float wmax[kComputeWarps][kHeads];
  float wsum[kComputeWarps][kHeads];
  alignas(8) uint64_t raw_full[kRawSlots];
  int grow[3], stop[3];
  int bad[kRawSlots];
  int abort_flag, poisoned;
  uint32_t new_words[kD / 8], new_sb[kD / 64];           // the new token's codes and (scale, bias) pairs (update-and-fetch)
};

__device__ inline float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ inline uint32_t f32x2_to_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ inline float2 h2_to_f2(uint32_t u) { return __half22float2(*reinterpret_cast<__half2*>(&u)); }
// two 16-bit numbers of the cache's scale / bias type as binary32
template <bool kBf>
__device__ __forceinline__ float2 pair_to_f2(uint32_t u) {
  if (kBf) return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}
__device__ inline void compute_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }   // the eight compute warps
// four 8x8 b16 matrices, each transposed; lane l supplies the address of row l % 8 of matrix l / 8; register i <-
// matrix i, thread (g, t) receiving the elements (rows 2t, 2t+1, column g)
__device__ inline void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}
__device__ inline void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <bool kBf>
__global__ void __launch_bounds__(kThreads, 1) decode_mla_codes_kernel(const __grid_constant__ MlaParams P) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  MlaSmem& sm = *reinterpret_cast<MlaSmem*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, a = blockIdx.y;
  const int n_rep = y.Hq;                                // one KV head

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- this CTA's share of the agent's keys (inputs no kernel writes) ----
  int n = P.kv_lens[a];
  const bool bad_len = n < 0 || n > P.len_cap;           // the host's bound on every length: the key shares cover that many keys
  if (bad_len) n = 0;
  const int lo = P.window > 0 ? max(0, n - P.window) : 0;
  const int b_lo = lo >> 6, b_hi = (n + 63) >> 6;        // 64-key blocks of the attended range
  const int b0 = min(b_hi, b_lo + split * P.blocks_per_split);
  const int n_iter = min(b_hi, b0 + P.blocks_per_split) - b0;
  float* rec = P.records + ((size_t)a * P.n_splits + split) * kHeads * kRecStride;
  if (n_iter <= 0) {
    // nothing to attend in this share: an empty record (the preceding kernels may still be reading the records)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x < kHeads) { rec[threadIdx.x * kRecStride + kDv] = -INFINITY; rec[threadIdx.x * kRecStride + kDv + 1] = 0.f; }
    if (bad_len && split == 0 && threadIdx.x == 0) raise_flag(P.flags, Q4KV_FLAG_BAD_LENGTH);
    return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRawSlots; ++s) { mbar_init(&sm.raw_full[s], 1); sm.bad[s] = 0; }
    for (int i = 0; i < 3; ++i) { sm.grow[i] = 0; sm.stop[i] = 0; }
    sm.abort_flag = 0; sm.poisoned = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();
  if (threadIdx.x < kRawSlots && threadIdx.x < n_iter)   // the first block-table entries, fetched towards the SM meanwhile
    asm volatile("prefetch.global.L1 [%0];" ::"l"(P.tables + (size_t)a * P.max_blocks + ((2 * (b0 + (int)threadIdx.x)) >> 3)) : "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the pool may still be being written by the preceding kernel
  volatile int* abort_flag = &sm.abort_flag;

  // Raw 64-key blocks: one bulk copy each into the ring, issued by thread 0 -- the first kRawSlots blocks here, block
  // j + kRawSlots once every warp has left block j's raw bytes (the barrier after the score step).
  auto issue_block = [&](int j) {
    const int r = j % kRawSlots;
    const int c = 2 * (b0 + j);
    const int blk = P.tables[(size_t)a * P.max_blocks + (c >> 3)];
    if (blk < 0 || blk >= P.n_blocks) {
      sm.bad[r] = 1;
      sm.poisoned = 1;
      raise_flag(P.flags, Q4KV_FLAG_BAD_BLOCK);
      mbar_arrive(&sm.raw_full[r]);
    } else {
      sm.bad[r] = 0;
      mbar_arrive_expect_tx(&sm.raw_full[r], kRawBytes);
      bulk_load(sm.raw[r], head_block(P.pool, y, P.layer, blk, 0) + (size_t)(c & 7) * kChunkBytes, kRawBytes, &sm.raw_full[r]);
    }
  };
  int issued = 0;                                        // thread 0: blocks whose copy has been issued
  if (threadIdx.x == 0) {
    issued = min(n_iter, kRawSlots);
    for (int j = 0; j < issued; ++j) issue_block(j);
  }

  // Update-and-fetch: the CTA whose share ends with the agent's last block quantizes the row of position n - 1
  // (one warp, while the first copies are in flight) and, once that block has landed, patches it in shared memory
  // and stores the same words to the pool.  No other CTA reads that block.
  const bool has_new = P.k_new != nullptr && b0 + n_iter == b_hi;
  if (has_new && warp == 0) {
#pragma unroll 1
    for (int base = 0; base < kD / 8; base += 32) {
      const int w = base + lane;
      float x[8];
      if (w < kD / 8) {
        load_eight_bf16(P.k_new, (size_t)a * kD + 8 * w, x);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = 0.f;
      }
      const QuantOut qo = quantize_eight(x, kBf);        // eight lanes per group of 64; 72 words = 9 whole groups
      if (w < kD / 8) {
        sm.new_words[w] = qo.word;
        if ((w & 7) == 0) sm.new_sb[w >> 3] = qo.sb;
      }
    }
  }

  const int tq = threadIdx.x;                            // 0..255
  const int g = lane >> 2, tid = lane & 3;               // fragment coordinates
  {
    // ---- stage the queries as A fragments: bf16 -> binary16 times a power of two per head.  Key word p of a lane
    // (elements 32 p + 8 tid + 0..7) feeds two products: (0,4 | 1,5) and (2,6 | 3,7); the second pair of each meets
    // codes one nibble up (a factor 16, divided out here).  Rows g and g + 8 of the operand are heads g and g + 8. ----
    const int h = tq >> 4, sub = tq & 15;                // sixteen consecutive lanes share a head; words sub, sub + 16, ...
    const bool live = h < n_rep;
    const uint16_t* qrow = P.q + ((size_t)a * y.Hq + (live ? h : 0)) * kD;
    uint4 v[5];
    float mx = 0.f, wsum[5];
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const int w = sub + 16 * k;
      v[k] = (live && w < kD / 8) ? *reinterpret_cast<const uint4*>(qrow + 8 * w) : make_uint4(0u, 0u, 0u, 0u);
      const uint32_t u[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
      float sum = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float xl = __uint_as_float(u[e] << 16), xh = __uint_as_float(u[e] & 0xffff0000u);
        mx = fmaxf(mx, fmaxf(fabsf(xl), fabsf(xh)));
        sum += xl + xh;
      }
      wsum[k] = sum;
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    // group sums: word sub + 16 k lies in group 2 k + sub / 8, whose eight words sit in eight consecutive lanes
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      float s = wsum[k];
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const int gi = 2 * k + (sub >> 3);
      if ((sub & 7) == 0 && gi < kG) sm.qsum[h][gi] = s * P.scale_log2;
    }
    int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
    if (mx == 0.f) ex = 0;
    ex = min(max(ex, -100), 100);
    const float sf = __uint_as_float((uint32_t)(127 + 11 - ex) << 23);        // 2048 <= max |q| * sf < 4096
    const float sl = sf * 0.0625f;
    if (sub == 0) sm.kappa[h] = P.scale_log2 * __uint_as_float((uint32_t)(127 + 13 + ex) << 23);   // 2^24 / sf
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const int w = sub + 16 * k;
      if (w >= kD / 8) continue;
      const uint32_t u01 = v[k].x, u23 = v[k].y, u45 = v[k].z, u67 = v[k].w;
      const float x0 = __uint_as_float(u01 << 16), x1 = __uint_as_float(u01 & 0xffff0000u);
      const float x2 = __uint_as_float(u23 << 16), x3 = __uint_as_float(u23 & 0xffff0000u);
      const float x4 = __uint_as_float(u45 << 16), x5 = __uint_as_float(u45 & 0xffff0000u);
      const float x6 = __uint_as_float(u67 << 16), x7 = __uint_as_float(u67 & 0xffff0000u);
      const int p = w >> 2, t = w & 3, row = h >> 3;     // row 0: registers a0, a2; row 1 (heads 8..15): a1, a3
      uint32_t* f0 = reinterpret_cast<uint32_t*>(&sm.qfrag[2 * p][(h & 7) * 4 + t]);
      uint32_t* f1 = reinterpret_cast<uint32_t*>(&sm.qfrag[2 * p + 1][(h & 7) * 4 + t]);
      f0[row] = f32x2_to_h2(x0 * sf, x4 * sf); f0[2 + row] = f32x2_to_h2(x1 * sl, x5 * sl);
      f1[row] = f32x2_to_h2(x2 * sf, x6 * sf); f1[2 + row] = f32x2_to_h2(x3 * sl, x7 * sl);
    }
  }
  compute_barrier();                                     // query fragments, group sums and kappa are complete

  // The queries never change: their A fragments (36 products x 4 registers) live in registers for the whole launch.
  uint32_t qa[kD / 16][4];
#pragma unroll
  for (int ks = 0; ks < kD / 16; ++ks) {
    const uint4 f = sm.qfrag[ks][lane];
    qa[ks][0] = f.x; qa[ks][1] = f.y; qa[ks][2] = f.z; qa[ks][3] = f.w;
  }
  float kap[2], m_ref[2], l_part[2], bias_acc[2];        // heads g and g + 8
  kap[0] = sm.kappa[g]; kap[1] = sm.kappa[g + 8];
  m_ref[0] = -INFINITY; m_ref[1] = -INFINITY; l_part[0] = 0.f; l_part[1] = 0.f; bias_acc[0] = 0.f; bias_acc[1] = 0.f;
  // value accumulators of group `warp`: o[k][nt]: dims of nibble k of every 16-bit element; heads 8 nt + 2 tid, + 1;
  // registers 0, 1: element row g (first half rows); 2, 3: element row g of the second half rows
  float o[4][2][4];
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) { o[k][nt][0] = 0.f; o[k][nt][1] = 0.f; o[k][nt][2] = 0.f; o[k][nt][3] = 0.f; }

  // score step: this warp's key tile is tile i = warp % 4 of chunk ci = warp / 4 (tokens 4 g + i of that chunk)
  const int ci = warp >> 2, ti = warp & 3;
  const uint32_t kc_at = ci * kChunkBytes + (ti * 576 + (g * 4 + tid) * 4) * 4;      // + j * 512 for piece j < 4
  const uint32_t kc_last = ci * kChunkBytes + (ti * 576 + 512 + (g * 4 + tid) * 2) * 4;
  const uint32_t sb_at = ci * kChunkBytes + 9216 + (ti * 4 + tid) * 72;              // 18 half2: token e = 0, 1 x 9 groups
  // value step: ldmatrix lane address (lane l: matrix l / 8 = (half row l/8 % 2, key tile parity l / 16), row l % 8)
  const uint32_t vre_lane = (uint32_t)(((warp * 8 + (lane >> 4)) * 2 + ((lane >> 3) & 1)) * 128 + (lane & 7) * 16);

  float m_o[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // the same references for the accumulators' heads 2 tid, 2 tid + 1 (+ 8)
  bool stopped = false;
  for (int j = 0; j < n_iter; ++j) {
    const int r = j % kRawSlots, b = j & 1;
    mbar_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots), abort_flag);     // a wait that runs out raises the give-up flag
    if (has_new && j == n_iter - 1) {
      // words 0..71 and the nine (scale, bias) pairs of position n - 1, one per thread
      if (sm.bad[r] == 0 && tq < kD / 8 + kD / 64) {
        const int tau_n = (n - 1) & 31, c = 2 * (b0 + j);
        const uint32_t at = (uint32_t)(((n - 1) >> 5) & 1) * kChunkBytes +
                            (tq < kD / 8 ? y.off_kc + 4u * k_word_offset(tau_n, tq, kG)
                                         : y.off_ksb + 4u * sb_offset(tau_n, tq - kD / 8, kG));
        const uint32_t val = tq < kD / 8 ? sm.new_words[tq] : sm.new_sb[tq - kD / 8];
        *reinterpret_cast<uint32_t*>(sm.raw[r] + at) = val;
        const int blk = P.tables[(size_t)a * P.max_blocks + (c >> 3)];      // checked when the copy was issued
        // the caller of the update-and-fetch entry owns the pool for writing
        uint8_t* dst = const_cast<uint8_t*>(head_block(P.pool, y, P.layer, blk, 0)) + (size_t)(c & 7) * kChunkBytes + at;
        *reinterpret_cast<uint32_t*>(dst) = val;
      }
      compute_barrier();
    }
    // =========== score step: this warp's key tile against all 16 heads, on the codes ===========
    const uint8_t* raw = sm.raw[r];
    const bool bad_blk = sm.bad[r] != 0;
    const int pos0 = (b0 + j) * 64 + ci * 32 + 8 * tid + ti;               // this lane's two tokens: pos0 and pos0 + 4
    const bool v0 = !bad_blk && pos0 >= lo && pos0 < n, v1 = !bad_blk && pos0 + 4 >= lo && pos0 + 4 < n;
    float lg[4];                                                           // logits (log2 units): head g: tokens 0, 1; head g + 8: tokens 0, 1
    uint32_t kw[18];
    {
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const uint4 t4 = *reinterpret_cast<const uint4*>(raw + kc_at + jj * 512);
        kw[4 * jj] = t4.x; kw[4 * jj + 1] = t4.y; kw[4 * jj + 2] = t4.z; kw[4 * jj + 3] = t4.w;
      }
      const uint2 t2 = *reinterpret_cast<const uint2*>(raw + kc_last);
      kw[16] = t2.x; kw[17] = t2.y;
      float sc[4] = {0.f, 0.f, 0.f, 0.f}, ub[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int gi = 0; gi < kG; ++gi) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i2 = 0; i2 < 2; ++i2) {
          const int p = 2 * gi + i2;
          const uint32_t w = kw[p], wh = w >> 8;
          mma_f16(acc, qa[2 * p][0], qa[2 * p][1], qa[2 * p][2], qa[2 * p][3], w & kMaskLo, w & kMaskHi);
          mma_f16(acc, qa[2 * p + 1][0], qa[2 * p + 1][1], qa[2 * p + 1][2], qa[2 * p + 1][3], wh & kMaskLo, wh & kMaskHi);
        }
        const float2 sb0 = sb_to_f2<kBf>(*reinterpret_cast<const uint32_t*>(raw + sb_at + 4 * gi));        // token 0: (scale, bias)
        const float2 sb1 = sb_to_f2<kBf>(*reinterpret_cast<const uint32_t*>(raw + sb_at + 36 + 4 * gi));   // token 1
        const float q0 = sm.qsum[g][gi], q1 = sm.qsum[g + 8][gi];
        sc[0] = fmaf(acc[0], sb0.x, sc[0]); sc[1] = fmaf(acc[1], sb1.x, sc[1]);
        sc[2] = fmaf(acc[2], sb0.x, sc[2]); sc[3] = fmaf(acc[3], sb1.x, sc[3]);
        ub[0] = fmaf(q0, sb0.y, ub[0]); ub[1] = fmaf(q0, sb1.y, ub[1]);
        ub[2] = fmaf(q1, sb0.y, ub[2]); ub[3] = fmaf(q1, sb1.y, ub[3]);
      }
      lg[0] = v0 ? fmaf(kap[0], sc[0], ub[0]) : -INFINITY; lg[1] = v1 ? fmaf(kap[0], sc[1], ub[1]) : -INFINITY;
      lg[2] = v0 ? fmaf(kap[1], sc[2], ub[2]) : -INFINITY; lg[3] = v1 ? fmaf(kap[1], sc[3], ub[3]) : -INFINITY;
    }
    // the key words again, regrouped for the value step: group gi's two words of this lane, 8 bytes
    {
      uint8_t* dst = sm.vre[b] + ((warp * 2 + (tid >> 1)) * 128 + g * 16 + (tid & 1) * 8);
#pragma unroll
      for (int gi = 0; gi < kGv; ++gi)
        *reinterpret_cast<uint2*>(dst + gi * (8 * 2 * 128)) = make_uint2(kw[2 * gi], kw[2 * gi + 1]);
    }
    // scales and biases of the lane's two tokens for the value step: lane g writes group g (dead tokens: zero)
    {
      const uint32_t e0 = v0 ? *reinterpret_cast<const uint32_t*>(raw + sb_at + 4 * g) : 0u;
      const uint32_t e1 = v1 ? *reinterpret_cast<const uint32_t*>(raw + sb_at + 36 + 4 * g) : 0u;
      sm.stab[b][g][warp][tid] = __byte_perm(e0, e1, 0x5410);
      sm.btab[b][g][warp][tid] = __byte_perm(e0, e1, 0x7632);
    }
    // probabilities against the current references; a block that outgrows them is redone below
    const float mx0 = fmaxf(lg[0], lg[1]), mx1 = fmaxf(lg[2], lg[3]);
    const bool grow = mx0 > m_ref[0] + kLazy || (m_ref[0] == -INFINITY && mx0 != -INFINITY) ||
                      mx1 > m_ref[1] + kLazy || (m_ref[1] == -INFINITY && mx1 != -INFINITY);
    if (__any_sync(0xffffffffu, grow) && lane == 0) sm.grow[j % 3] = 1;
    float p0 = v0 ? fast_exp2(lg[0] - m_ref[0]) : 0.f, p1 = v1 ? fast_exp2(lg[1] - m_ref[0]) : 0.f;
    float p2 = v0 ? fast_exp2(lg[2] - m_ref[1]) : 0.f, p3 = v1 ? fast_exp2(lg[3] - m_ref[1]) : 0.f;
    sm.ptile[b][warp][0][lane] = make_float2(p0, p1);
    sm.ptile[b][warp][1][lane] = make_float2(p2, p3);
    if (tq == 0) sm.stop[j % 3] = *abort_flag;           // sampled by one thread: all 256 leave in the same block
    compute_barrier();                                   // the block's words, tables and probabilities are in place; the raw slot is free
    if (sm.stop[j % 3]) { stopped = true; break; }
    if (tq == 0) {
      sm.grow[(j + 2) % 3] = 0;                          // not touched again before the barrier after next
      if (j + kRawSlots < n_iter) { issue_block(j + kRawSlots); issued = j + kRawSlots + 1; }
    }
    if (sm.grow[j % 3]) {
      // ---- exact per-head maxima of the block become the references; what has been accumulated is rescaled and the
      // block's probabilities are retaken ----
      float w0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)), w1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      w0 = fmaxf(w0, __shfl_xor_sync(0xffffffffu, w0, 2)); w1 = fmaxf(w1, __shfl_xor_sync(0xffffffffu, w1, 2));
      if (tid == 0) { sm.wmax[warp][g] = w0; sm.wmax[warp][g + 8] = w1; }
      compute_barrier();
      auto new_ref = [&](int head, float old) {
        float m_new = old;
#pragma unroll
        for (int w = 0; w < kComputeWarps; ++w) m_new = fmaxf(m_new, sm.wmax[w][head]);
        return m_new;
      };
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float m_new = new_ref(g + 8 * e, m_ref[e]);
        const float f = m_new == -INFINITY ? 1.f : fast_exp2(m_ref[e] - m_new);      // m_ref = -inf: 0
        l_part[e] *= f; bias_acc[e] *= f;
        m_ref[e] = m_new;
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int head = 2 * tid + (x & 1) + 8 * (x >> 1);
        const float m_new = new_ref(head, m_o[x]);
        const float f = m_new == -INFINITY ? 1.f : fast_exp2(m_o[x] - m_new);
        m_o[x] = m_new;
#pragma unroll
        for (int k = 0; k < 4; ++k) { o[k][x >> 1][x & 1] *= f; o[k][x >> 1][2 + (x & 1)] *= f; }
      }
      p0 = v0 ? fast_exp2(lg[0] - m_ref[0]) : 0.f; p1 = v1 ? fast_exp2(lg[1] - m_ref[0]) : 0.f;
      p2 = v0 ? fast_exp2(lg[2] - m_ref[1]) : 0.f; p3 = v1 ? fast_exp2(lg[3] - m_ref[1]) : 0.f;
      sm.ptile[b][warp][0][lane] = make_float2(p0, p1);
      sm.ptile[b][warp][1][lane] = make_float2(p2, p3);
      compute_barrier();
    }
    l_part[0] += p0 + p1; l_part[1] += p2 + p3;

    // =========== value step: the 64 dims of group `warp`, all 64 keys of the block, on the codes ===========
    {
      const uint32_t vbase = smem_u32(sm.vre[b]) + vre_lane;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        uint32_t R[4];
        ldmatrix_x4_trans(R, vbase + ks * 512);
        uint32_t Bh[2][2], Bl[2][2];                     // [heads 0-7 | 8-15][key tile 2 ks | 2 ks + 1]: p * s as hi + lo
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float2 ss = pair_to_f2<kBf>(sm.stab[b][warp][2 * ks + hf][tid]);
          const float2 bb = pair_to_f2<kBf>(sm.btab[b][warp][2 * ks + hf][tid]);
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const float2 pf = sm.ptile[b][2 * ks + hf][nt][lane];
            const float w0 = pf.x * ss.x, w1 = pf.y * ss.y;
            Bh[nt][hf] = f32x2_to_h2(w0, w1);
            const float2 hi = h2_to_f2(Bh[nt][hf]);
            Bl[nt][hf] = f32x2_to_h2(w0 - hi.x, w1 - hi.y);
            bias_acc[nt] = fmaf(pf.x, bb.x, fmaf(pf.y, bb.y, bias_acc[nt]));
          }
        }
        uint32_t Rh[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) Rh[i] = R[i] >> 8;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          mma_f16(o[0][nt], R[0] & kMaskLo, R[1] & kMaskLo, R[2] & kMaskLo, R[3] & kMaskLo, Bh[nt][0], Bh[nt][1]);
          mma_f16(o[1][nt], R[0] & kMaskHi, R[1] & kMaskHi, R[2] & kMaskHi, R[3] & kMaskHi, Bh[nt][0], Bh[nt][1]);
          mma_f16(o[2][nt], Rh[0] & kMaskLo, Rh[1] & kMaskLo, Rh[2] & kMaskLo, Rh[3] & kMaskLo, Bh[nt][0], Bh[nt][1]);
          mma_f16(o[3][nt], Rh[0] & kMaskHi, Rh[1] & kMaskHi, Rh[2] & kMaskHi, Rh[3] & kMaskHi, Bh[nt][0], Bh[nt][1]);
          mma_f16(o[0][nt], R[0] & kMaskLo, R[1] & kMaskLo, R[2] & kMaskLo, R[3] & kMaskLo, Bl[nt][0], Bl[nt][1]);
          mma_f16(o[1][nt], R[0] & kMaskHi, R[1] & kMaskHi, R[2] & kMaskHi, R[3] & kMaskHi, Bl[nt][0], Bl[nt][1]);
          mma_f16(o[2][nt], Rh[0] & kMaskLo, Rh[1] & kMaskLo, Rh[2] & kMaskLo, Rh[3] & kMaskLo, Bl[nt][0], Bl[nt][1]);
          mma_f16(o[3][nt], Rh[0] & kMaskHi, Rh[1] & kMaskHi, Rh[2] & kMaskHi, Rh[3] & kMaskHi, Bl[nt][0], Bl[nt][1]);
        }
      }
    }
  }

  // ---- this share's record: acc[16][512] (unnormalised, relative to m), m, l ----
  compute_barrier();                                     // every warp has left the loop: the small arrays can be reused
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float lh = l_part[e], bh = bias_acc[e];
    lh += __shfl_xor_sync(0xffffffffu, lh, 1); bh += __shfl_xor_sync(0xffffffffu, bh, 1);
    lh += __shfl_xor_sync(0xffffffffu, lh, 2); bh += __shfl_xor_sync(0xffffffffu, bh, 2);
    if (tid == 0) { sm.wsum[warp][g + 8 * e] = lh; sm.wmax[warp][g + 8 * e] = bh; }   // wmax: this warp's group's bias sums
  }
  compute_barrier();
  const bool spoiled = stopped || sm.poisoned != 0;
  if (stopped && tq == 0) {
    // giving up: let the copies that may still be in flight land before shared memory is released
    for (int jj = max(0, issued - kRawSlots); jj < issued; ++jj)
      for (uint32_t i = 0; i < 64 && !mbar_try_wait(&sm.raw_full[jj % kRawSlots], (uint32_t)(jj / kRawSlots) & 1u); ++i) {}
    raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
  }
  // accumulator (k, nt, register cr): head 8 nt + 2 tid + cr % 2; 16-bit element column g of half row cr / 2, nibble k:
  // word p = 2 warp + (g / 2) % 2 of source lane tid 2 (cr / 2) + g / 4, half g % 2 -> dim 32 p + 8 tid_src + 4 (g % 2) + k
#pragma unroll
  for (int nt = 0; nt < 2; ++nt)
#pragma unroll
    for (int cr = 0; cr < 4; ++cr) {
      const int head = 8 * nt + 2 * tid + (cr & 1);
      const float bias = sm.wmax[warp][head];
      const int d_base = 32 * (2 * warp + ((g >> 1) & 1)) + 8 * (2 * (cr >> 1) + (g >> 2)) + 4 * (g & 1);
      float4 v;
      v.x = fmaf(o[0][nt][cr], 16777216.f, bias); v.y = fmaf(o[1][nt][cr], 1048576.f, bias);   // 2^24; 2^24 / 16
      v.z = fmaf(o[2][nt][cr], 16777216.f, bias); v.w = fmaf(o[3][nt][cr], 1048576.f, bias);
      if (spoiled) v = make_float4(0.f, 0.f, 0.f, 0.f);
      float* at = rec + head * kRecStride + d_base;      // records are 8-byte aligned (514 floats per head)
      *reinterpret_cast<float2*>(at) = make_float2(v.x, v.y);
      *reinterpret_cast<float2*>(at + 2) = make_float2(v.z, v.w);
    }
  if (warp == 0 && tid == 0) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int h = g + 8 * e;
      float lsum = 0.f;
#pragma unroll
      for (int w = 0; w < kComputeWarps; ++w) lsum += sm.wsum[w][h];
      rec[h * kRecStride + kDv] = spoiled ? -INFINITY : m_ref[e];
      rec[h * kRecStride + kDv + 1] = spoiled ? -1.f : lsum;               // negative: poisoned
    }
  }
}

}  // namespace

cudaError_t launch_mla_codes_kernel(const MlaDecodeParams& P, cudaStream_t st) {
  static bool configured[64][2] = {};
  const size_t smem = sizeof(MlaSmem);
  const int bf = P.y.sb_bf16 ? 1 : 0;
  void (*kernel)(const MlaParams) = bf ? decode_mla_codes_kernel<true> : decode_mla_codes_kernel<false>;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev][bf]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev][bf] = true;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P.n_splits, P.n_agents);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, P);
}

}  // namespace q4kv
