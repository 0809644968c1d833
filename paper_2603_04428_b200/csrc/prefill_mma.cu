// q4kv_prefill_attention, tensor-core path on the codes (d_qk = d_v in {128, 256}, at most four query heads per KV
// head): the queries of a new phase over the cached Q4 prefix plus the causal new tokens, all read from the Q4 cache
// in place (Sections 3.4 "chunked prefill" and 3.5 "cross-phase context injection"; GQA and sliding windows:
// Section 3.6).
//
// Flash-attention structure with the arithmetic on the 4-bit codes (no dequantized tile is ever built): a CTA owns a
// run of consecutive queries of one agent for the query heads of one KV head and walks the 32-token chunks of that
// pair's keys through a shared-memory ring filled by bulk asynchronous copies.  Its eight warps are (head slot, query
// sub-tile) pairs -- 4 x 2, 2 x 4 or 1 x 8 by the number of query heads per KV head -- with two 16-row tiles per warp at
// d = 128 and one at d = 256 (where a tile's accumulators are 128 registers per lane).
//   * Scores: mma.sync m16n8k16 f16.  A 16-bit lane holding a code c in its low nibble IS the binary16 subnormal
//     c * 2^-24, so the key operand is the packed word under a mask (nibble 1 of a lane carries a factor 16 that the
//     matching query elements are divided by); every bf16 query row is scaled by a power of two into binary16 without
//     rounding.  (The 8-bit float forms of mma.sync cost two f16 tensor instructions plus conversions and adds on this
//     part, so they are not used.)  Per 64-element group the integer dot product is scaled by the token's scale, and the
//     token's bias meets the row's per-group query sum.
//   * Values: mma.sync m16n8k16 f16 with the value codes as binary16 subnormals c * 2^-24 (masked in place from the
//     token-packed words) and probabilities pre-multiplied by the token's group scale, carried as a two-term binary16
//     sum (two products per value tile), so the value product is good to ~2^-22 of the cached magnitudes; the bias
//     part is a per-row float32 scalar sum.
//   * The score fragment of two adjacent key tiles is the A fragment of the value product, as in any
//     register-resident flash attention, so probabilities never leave their lane.
// Measured: 146 TFLOP/s on 8 x (8192 + 1024) tokens at d = 128 with 32 / 8 heads; 148 TFLOP/s on 8 x (4096 + 512)
// tokens at d = 256 with 16 / 8 heads.
#include "q4kv_layout.cuh"
#include "quantize_core.cuh"

namespace q4kv {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kSlots = 16;                 // ring depth in chunks
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kMaskLo = 0x000F000Fu, kMaskHi = 0x00F000F0u;

__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ inline void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_arrive(uint64_t* bar) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ inline bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ inline void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ inline void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline void mma_f16(float (&c)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
__device__ inline float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ inline float2 h2_to_f2(uint32_t u) { return __half22float2(*reinterpret_cast<__half2*>(&u)); }
__device__ inline uint32_t f32x2_to_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
struct PrefillParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks;
  const int32_t* tables;
  const int32_t* kv_lens;
  const int32_t* q_offs;
  int window;
  const uint16_t* q;          // bf16 [total_q][Hq][D]
  float scale_log2;
  void* out;
  int out_dtype;
  float* lse;
  int32_t* flags;
};

template <int R, int G>
struct PrefillSmem {
  static constexpr int kChunkBytes = 2304 * G;           // 32 * (32 G + 4 G) * 2: 4608 at d = 128, 9216 at d = 256
  static constexpr int kRows = kWarps * R * 16;
  alignas(128) uint8_t ring[kSlots * kChunkBytes];
  alignas(16) uint4 qfrag[kWarps][R][2 * G][2][32];      // [warp][row tile][key word][half of the word][lane] = A registers
  float kappa[kRows];                                    // scale_log2 * 2^(ex + 13) of each row
  float qsum[kRows][G];                                  // scale_log2 * per-group sums of the true query row
  alignas(8) uint64_t full[kSlots];
  int released[kSlots];                                  // warps that have finished with each slot (monotonic)
  int bad[kSlots];
  int abort_flag;
};

template <int R, int G, bool kBf>
__global__ void __launch_bounds__(kThreads, 1) prefill_mma_kernel(const __grid_constant__ PrefillParams P) {
  constexpr int D = 64 * G, Dv = D;
  constexpr int kRowWords = D / 8;                       // 16 or 32: the words of a query row sit in that many consecutive lanes
  using S = PrefillSmem<R, G>;
  constexpr int kChunkBytes = S::kChunkBytes;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  S& sm = *reinterpret_cast<S*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tid = lane & 3;
  const int qt = blockIdx.x, hk = blockIdx.y, a = blockIdx.z;
  const int n_rep = y.n_rep;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.full[s], 1); sm.released[s] = 0; sm.bad[s] = 0; }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // ---- this CTA's queries and key range ----
  const int q0 = P.q_offs[a], q_len = P.q_offs[a + 1] - q0;
  const int kv_len = P.kv_lens[a];
  // the eight warps are (head slot, query sub-tile) pairs: 4 x 2 for three or four query heads per KV head, 2 x 4 for
  // two, 1 x 8 for one, so that no warp works on a head that does not exist
  const int hs = n_rep > 2 ? 4 : n_rep;
  const int tile_q = (kWarps / hs) * 16 * R;             // queries per CTA
  const int i_min = qt * tile_q;
  if (i_min >= q_len) return;                            // uniform: no thread has passed a barrier yet
  const bool bad_len = kv_len < 0 || kv_len > P.max_blocks * kBlockTokens || q_len > kv_len;
  if (bad_len && threadIdx.x == 0) raise_flag(P.flags, Q4KV_FLAG_BAD_LENGTH);
  const int i_max = min(q_len, i_min + tile_q) - 1;
  const int prefix = kv_len - q_len;                     // query i sits at position prefix + i
  const int c_end = bad_len ? 0 : (prefix + i_max) / 32 + 1;
  const int c_begin = (bad_len || P.window == 0) ? 0 : max(0, prefix + i_min - P.window + 1) >> 5;
  const int n_chunks = max(0, c_end - c_begin);
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the new chunk was appended by the preceding kernel

  // Chunk k of this CTA goes to slot k % kSlots; issued by one thread.
  auto issue = [&](int k) {
    const int c = c_begin + k, slot = k % kSlots;
    const int blk = P.tables[(size_t)a * P.max_blocks + (c >> 3)];
    if (blk < 0 || blk >= P.n_blocks) {
      sm.bad[slot] = 1;
      raise_flag(P.flags, Q4KV_FLAG_BAD_BLOCK);
      mbar_arrive(&sm.full[slot]);
    } else {
      sm.bad[slot] = 0;
      mbar_arrive_expect_tx(&sm.full[slot], kChunkBytes);
      bulk_load(sm.ring + (size_t)slot * kChunkBytes,
                head_block(P.pool, y, P.layer, blk, hk) + (size_t)(c & 7) * kChunkBytes, kChunkBytes, &sm.full[slot]);
    }
  };
  if (warp == 0 && lane < kSlots && lane < n_chunks) issue(lane);

  // ---- stage the query rows: binary16 in A-fragment order, per-row factor and group sums ----
  for (int item = threadIdx.x; item < S::kRows * kRowWords; item += kThreads) {
    const int row = item / kRowWords, w = item % kRowWords;
    const int wv = row / (16 * R), rt = (row >> 4) % R, rr = row & 15;
    const int h = wv % hs, qhalf = wv / hs;
    const int i = i_min + (qhalf * R + rt) * 16 + rr;
    const bool valid = i < q_len && h < n_rep && !bad_len;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (valid) v = *reinterpret_cast<const uint4*>(P.q + ((size_t)(q0 + i) * y.Hq + (size_t)hk * n_rep + h) * D + 8 * w);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
    float x[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) { x[2 * j] = __uint_as_float(u[j] << 16); x[2 * j + 1] = __uint_as_float(u[j] & 0xffff0000u); }
    float mx = 0.f, sum = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) { mx = fmaxf(mx, fabsf(x[j])); sum += x[j]; }
#pragma unroll
    for (int o = kRowWords / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));   // the lanes of a row
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);           // 8 words per group
    int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
    if (mx == 0.f) ex = 0;
    ex = min(max(ex, -100), 100);
    const float sf = __uint_as_float((uint32_t)(127 + 11 - ex) << 23);                     // 2048 <= max |q| * sf < 4096
    const float sl = sf * 0.0625f;                       // elements that meet a code in nibble 1 of its 16-bit lane
    // Key word w of a token holds elements 8w..8w+7; its two 16x8x16 products take, per lane,
    // (0,4 | 1,5) and (2,6 | 3,7): registers a0/a1 = rows g/g+8 of the first pair, a2/a3 of the second.
    const int ks = w >> 2, dl = (rr & 7) * 4 + (w & 3), up = rr >> 3;
    uint32_t* f1 = reinterpret_cast<uint32_t*>(&sm.qfrag[wv][rt][ks][0][dl]);
    uint32_t* f2 = reinterpret_cast<uint32_t*>(&sm.qfrag[wv][rt][ks][1][dl]);
    f1[up] = f32x2_to_h2(x[0] * sf, x[4] * sf); f1[2 + up] = f32x2_to_h2(x[1] * sl, x[5] * sl);
    f2[up] = f32x2_to_h2(x[2] * sf, x[6] * sf); f2[2 + up] = f32x2_to_h2(x[3] * sl, x[7] * sl);
    if ((w & 7) == 0) sm.qsum[row][w >> 3] = sum * P.scale_log2;
    if (w == 0) sm.kappa[row] = P.scale_log2 * __uint_as_float((uint32_t)(127 + 13 + ex) << 23);
  }
  __syncthreads();

  // ---- per-warp rows: head h, R tiles of 16 consecutive queries; a lane owns rows g and g+8 of each tile ----
  const int h = warp % hs, qhalf = warp / hs;
  float kap[R][2], qs[R][2][G], m_run[R][2], l_e[R][2], l_o[R][2], bias_e[R][2][G], bias_o[R][2][G];
  float o[R][Dv / 8][4];
#pragma unroll
  for (int rt = 0; rt < R; ++rt) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int row = (warp * R + rt) * 16 + g + 8 * r;
      kap[rt][r] = sm.kappa[row];
      m_run[rt][r] = -INFINITY; l_e[rt][r] = 0.f; l_o[rt][r] = 0.f;
#pragma unroll
      for (int gi = 0; gi < G; ++gi) { qs[rt][r][gi] = sm.qsum[row][gi]; bias_e[rt][r][gi] = 0.f; bias_o[rt][r][gi] = 0.f; }
    }
#pragma unroll
    for (int nt = 0; nt < Dv / 8; ++nt) { o[rt][nt][0] = 0.f; o[rt][nt][1] = 0.f; o[rt][nt][2] = 0.f; o[rt][nt][3] = 0.f; }
  }
  bool aborted = false, poisoned = false;
  const int W = P.window;

  for (int k = 0; k < n_chunks; ++k) {
    const int slot = k % kSlots, round = k / kSlots;
    if (aborted || !mbar_wait(&sm.full[slot], (uint32_t)round & 1u, &sm.abort_flag)) { aborted = true; break; }
    if (sm.bad[slot]) {
      poisoned = true;
    } else {
      const uint8_t* chunk = sm.ring + (size_t)slot * kChunkBytes;
      const uint4* kc4 = reinterpret_cast<const uint4*>(chunk);
      const uint4* ksb4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2));
      const uint4* vc4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2) + 128 * G);
      const uint4* vsb4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2) + 128 * G + 32 * (Dv / 2));
      const int pos0 = (c_begin + k) * 32;
      const bool tail = pos0 + 32 > kv_len;              // slots past the cache end may hold stale bytes

      // Two forms of the same step.  d = 128 (two 16-row tiles per warp): all groups' operands of the value product
      // are built first.  d = 256 (one tile per warp, 128 accumulator registers per lane): keys and values are taken
      // two groups and one group at a time, which keeps the live registers within the file.
      if (G == 2) {
        uint32_t apv[R][G][2][4], apl[R][G][2][4];         // value-product A operands, high and low term: [tile][group][MMA][register]
        bool active[R];
  #pragma unroll
        for (int rt = 0; rt < R; ++rt) {
          const int pq_lo = prefix + i_min + (qhalf * R + rt) * 16, pq_hi = pq_lo + 15;
          active[rt] = pos0 <= pq_hi && (W == 0 || pos0 + 31 > pq_lo - W);
          if (!active[rt]) continue;
          const bool need_mask = pos0 + 31 > pq_lo || (W > 0 && pos0 <= pq_hi - W);
          // ---- integer dot products per key tile and group ----
          float acc[4][G][4];
  #pragma unroll
          for (int i = 0; i < 4; ++i)
  #pragma unroll
            for (int gi = 0; gi < G; ++gi) { acc[i][gi][0] = 0.f; acc[i][gi][1] = 0.f; acc[i][gi][2] = 0.f; acc[i][gi][3] = 0.f; }
          uint4 kw[4];
  #pragma unroll
          for (int i = 0; i < 4; ++i) kw[i] = kc4[(i * 8 + g) * 4 + tid];
  #pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint4 a1 = sm.qfrag[warp][rt][ks][0][lane], a2 = sm.qfrag[warp][rt][ks][1][lane];
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t w = ks == 0 ? kw[i].x : ks == 1 ? kw[i].y : ks == 2 ? kw[i].z : kw[i].w;
              const uint32_t wh = w >> 8;
              mma_f16(acc[i][ks >> 1], a1, w & kMaskLo, w & kMaskHi);
              mma_f16(acc[i][ks >> 1], a2, wh & kMaskLo, wh & kMaskHi);
            }
          }
          // ---- scores in log2 units, mask, online softmax ----
          float s[4][2][2];                                // [tile][token e][row r]
  #pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 sb = ksb4[i * 4 + tid];
            const float2 e0g0 = sb_to_f2<kBf>(sb.x), e0g1 = sb_to_f2<kBf>(sb.y), e1g0 = sb_to_f2<kBf>(sb.z), e1g1 = sb_to_f2<kBf>(sb.w);
  #pragma unroll
            for (int r = 0; r < 2; ++r) {
              const float t0 = fmaf(acc[i][1][2 * r], e0g1.x, acc[i][0][2 * r] * e0g0.x);
              const float t1 = fmaf(acc[i][1][2 * r + 1], e1g1.x, acc[i][0][2 * r + 1] * e1g0.x);
              const float u0 = fmaf(qs[rt][r][1], e0g1.y, qs[rt][r][0] * e0g0.y);
              const float u1 = fmaf(qs[rt][r][1], e1g1.y, qs[rt][r][0] * e1g0.y);
              s[i][0][r] = fmaf(kap[rt][r], t0, u0);
              s[i][1][r] = fmaf(kap[rt][r], t1, u1);
            }
          }
          if (need_mask) {
  #pragma unroll
            for (int r = 0; r < 2; ++r) {
              const int pq = pq_lo + g + 8 * r;
  #pragma unroll
              for (int i = 0; i < 4; ++i)
  #pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const int pos = pos0 + 8 * tid + 4 * e + i;
                  if (pos > pq || (W > 0 && pos <= pq - W)) s[i][e][r] = -INFINITY;
                }
            }
          }
          float corr[2];
  #pragma unroll
          for (int r = 0; r < 2; ++r) {
            float cm = fmaxf(fmaxf(fmaxf(s[0][0][r], s[0][1][r]), fmaxf(s[1][0][r], s[1][1][r])),
                             fmaxf(fmaxf(s[2][0][r], s[2][1][r]), fmaxf(s[3][0][r], s[3][1][r])));
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
            float m_new = fmaxf(m_run[rt][r], cm);
            if (m_new == -INFINITY) m_new = 0.f;
            corr[r] = fast_exp2(m_run[rt][r] - m_new);
            m_run[rt][r] = m_new;
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float off = (i & 1) ? m_new + 4.f : m_new;   // odd tiles: p / 16 (their value codes carry a factor 16)
              s[i][0][r] = fast_exp2(s[i][0][r] - off);
              s[i][1][r] = fast_exp2(s[i][1][r] - off);
            }
            l_e[rt][r] = fmaf(l_e[rt][r], corr[r], (s[0][0][r] + s[0][1][r]) + (s[2][0][r] + s[2][1][r]));
            l_o[rt][r] = fmaf(l_o[rt][r], corr[r], (s[1][0][r] + s[1][1][r]) + (s[3][0][r] + s[3][1][r]));
          }
          if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
  #pragma unroll
            for (int gi = 0; gi < G; ++gi) {
              bias_e[rt][0][gi] *= corr[0]; bias_o[rt][0][gi] *= corr[0];
              bias_e[rt][1][gi] *= corr[1]; bias_o[rt][1][gi] *= corr[1];
            }
  #pragma unroll
            for (int nt = 0; nt < Dv / 8; ++nt) {
              o[rt][nt][0] *= corr[0]; o[rt][nt][1] *= corr[0]; o[rt][nt][2] *= corr[1]; o[rt][nt][3] *= corr[1];
            }
          }
          // ---- p * s_v per group as a two-term binary16 sum (high part + rounded remainder): the A operands of the
          // value product, which is then good to ~2^-22 whatever the magnitude of the cached values ----
  #pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 sb = vsb4[i * 4 + tid];
            float2 v[2][G] = {{sb_to_f2<kBf>(sb.x), sb_to_f2<kBf>(sb.y)}, {sb_to_f2<kBf>(sb.z), sb_to_f2<kBf>(sb.w)}};   // [e][group] = (scale, bias)
            if (tail) {
  #pragma unroll
              for (int e = 0; e < 2; ++e)
                if (pos0 + 8 * tid + 4 * e + i >= kv_len) { v[e][0] = make_float2(0.f, 0.f); v[e][1] = make_float2(0.f, 0.f); }
            }
  #pragma unroll
            for (int gi = 0; gi < G; ++gi)
  #pragma unroll
              for (int r = 0; r < 2; ++r) {
                const float x0 = s[i][0][r] * v[0][gi].x, x1 = s[i][1][r] * v[1][gi].x;
                const uint32_t hi = f32x2_to_h2(x0, x1);
                const float2 hf = h2_to_f2(hi);
                apv[rt][gi][i >> 1][(i & 1) * 2 + r] = hi;
                apl[rt][gi][i >> 1][(i & 1) * 2 + r] = f32x2_to_h2(x0 - hf.x, x1 - hf.y);
                const float b = fmaf(s[i][0][r], v[0][gi].y, s[i][1][r] * v[1][gi].y);
                if (i & 1) bias_o[rt][r][gi] += b; else bias_e[rt][r][gi] += b;
              }
          }
        }
        // ---- value product on the codes ----
        bool any_active = false;
  #pragma unroll
        for (int rt = 0; rt < R; ++rt) any_active |= active[rt];
        if (any_active) {
  #pragma unroll
          for (int q4 = 0; q4 < Dv / 32; ++q4) {
            const uint4 w4 = vc4[(q4 * 8 + g) * 4 + tid];
            const uint32_t wd[4] = {w4.x, w4.y, w4.z, w4.w};
            const int gi = q4 >> 1;
  #pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t wh = wd[j] >> 8;
              const uint32_t be0 = wd[j] & kMaskLo, be1 = wd[j] & kMaskHi, bo0 = wh & kMaskLo, bo1 = wh & kMaskHi;
  #pragma unroll
              for (int rt = 0; rt < R; ++rt) {
                if (!active[rt]) continue;
                mma_f16(o[rt][4 * q4 + j], apv[rt][gi][0], be0, be1);
                mma_f16(o[rt][4 * q4 + j], apv[rt][gi][1], bo0, bo1);
                mma_f16(o[rt][4 * q4 + j], apl[rt][gi][0], be0, be1);
                mma_f16(o[rt][4 * q4 + j], apl[rt][gi][1], bo0, bo1);
              }
            }
          }
        }
      } else {
        float prob[R][4][2][2];                            // probabilities of the active tiles: [tile][key tile][token e][row r]
        bool active[R];
  #pragma unroll
        for (int rt = 0; rt < R; ++rt) {
          const int pq_lo = prefix + i_min + (qhalf * R + rt) * 16, pq_hi = pq_lo + 15;
          active[rt] = pos0 <= pq_hi && (W == 0 || pos0 + 31 > pq_lo - W);
          if (!active[rt]) continue;
          const bool need_mask = pos0 + 31 > pq_lo || (W > 0 && pos0 <= pq_hi - W);
          // ---- integer dot products per key tile and group, two groups (one 16-byte piece per token row) at a time;
          // the token's scale meets them, its bias the per-group query sums ----
          float tsum[4][2][2], usum[4][2][2];              // [key tile][token e][row r]
  #pragma unroll
          for (int i = 0; i < 4; ++i)
  #pragma unroll
            for (int e = 0; e < 2; ++e) { tsum[i][e][0] = 0.f; tsum[i][e][1] = 0.f; usum[i][e][0] = 0.f; usum[i][e][1] = 0.f; }
  #pragma unroll
          for (int half = 0; half < G / 2; ++half) {
            float acc[4][2][4];
  #pragma unroll
            for (int i = 0; i < 4; ++i)
  #pragma unroll
              for (int gi = 0; gi < 2; ++gi) { acc[i][gi][0] = 0.f; acc[i][gi][1] = 0.f; acc[i][gi][2] = 0.f; acc[i][gi][3] = 0.f; }
            uint4 kw[4];
  #pragma unroll
            for (int i = 0; i < 4; ++i) kw[i] = kc4[i * 16 * G + half * 32 + g * 4 + tid];
  #pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint4 a1 = sm.qfrag[warp][rt][4 * half + ks][0][lane], a2 = sm.qfrag[warp][rt][4 * half + ks][1][lane];
  #pragma unroll
              for (int i = 0; i < 4; ++i) {
                const uint32_t w = ks == 0 ? kw[i].x : ks == 1 ? kw[i].y : ks == 2 ? kw[i].z : kw[i].w;
                const uint32_t wh = w >> 8;
                mma_f16(acc[i][ks >> 1], a1, w & kMaskLo, w & kMaskHi);
                mma_f16(acc[i][ks >> 1], a2, wh & kMaskLo, wh & kMaskHi);
              }
            }
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              // (scale, bias) of tokens e = 0, 1 for the groups 2 half and 2 half + 1
              float2 f[2][2];
              if (G == 2) {
                const uint4 sb = ksb4[i * 4 + tid];
                f[0][0] = sb_to_f2<kBf>(sb.x); f[0][1] = sb_to_f2<kBf>(sb.y); f[1][0] = sb_to_f2<kBf>(sb.z); f[1][1] = sb_to_f2<kBf>(sb.w);
              } else {
  #pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const uint4 sb = ksb4[(i * 4 + tid) * 2 + e];
                  f[e][0] = sb_to_f2<kBf>(half == 0 ? sb.x : sb.z); f[e][1] = sb_to_f2<kBf>(half == 0 ? sb.y : sb.w);
                }
              }
  #pragma unroll
              for (int e = 0; e < 2; ++e)
  #pragma unroll
                for (int r = 0; r < 2; ++r) {
                  tsum[i][e][r] = fmaf(acc[i][1][2 * r + e], f[e][1].x, fmaf(acc[i][0][2 * r + e], f[e][0].x, tsum[i][e][r]));
                  usum[i][e][r] = fmaf(qs[rt][r][2 * half + 1], f[e][1].y, fmaf(qs[rt][r][2 * half], f[e][0].y, usum[i][e][r]));
                }
            }
          }
          // ---- scores in log2 units, mask, online softmax ----
          float (&sc)[4][2][2] = prob[rt];
  #pragma unroll
          for (int i = 0; i < 4; ++i)
  #pragma unroll
            for (int e = 0; e < 2; ++e)
  #pragma unroll
              for (int r = 0; r < 2; ++r) sc[i][e][r] = fmaf(kap[rt][r], tsum[i][e][r], usum[i][e][r]);
          if (need_mask) {
  #pragma unroll
            for (int r = 0; r < 2; ++r) {
              const int pq = pq_lo + g + 8 * r;
  #pragma unroll
              for (int i = 0; i < 4; ++i)
  #pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const int pos = pos0 + 8 * tid + 4 * e + i;
                  if (pos > pq || (W > 0 && pos <= pq - W)) sc[i][e][r] = -INFINITY;
                }
            }
          }
          float corr[2];
  #pragma unroll
          for (int r = 0; r < 2; ++r) {
            float cm = fmaxf(fmaxf(fmaxf(sc[0][0][r], sc[0][1][r]), fmaxf(sc[1][0][r], sc[1][1][r])),
                             fmaxf(fmaxf(sc[2][0][r], sc[2][1][r]), fmaxf(sc[3][0][r], sc[3][1][r])));
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
            cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
            float m_new = fmaxf(m_run[rt][r], cm);
            if (m_new == -INFINITY) m_new = 0.f;
            corr[r] = fast_exp2(m_run[rt][r] - m_new);
            m_run[rt][r] = m_new;
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float off = (i & 1) ? m_new + 4.f : m_new;   // odd tiles: p / 16 (their value codes carry a factor 16)
              sc[i][0][r] = fast_exp2(sc[i][0][r] - off);
              sc[i][1][r] = fast_exp2(sc[i][1][r] - off);
            }
            l_e[rt][r] = fmaf(l_e[rt][r], corr[r], (sc[0][0][r] + sc[0][1][r]) + (sc[2][0][r] + sc[2][1][r]));
            l_o[rt][r] = fmaf(l_o[rt][r], corr[r], (sc[1][0][r] + sc[1][1][r]) + (sc[3][0][r] + sc[3][1][r]));
          }
          if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
  #pragma unroll
            for (int gi = 0; gi < G; ++gi) {
              bias_e[rt][0][gi] *= corr[0]; bias_o[rt][0][gi] *= corr[0];
              bias_e[rt][1][gi] *= corr[1]; bias_o[rt][1][gi] *= corr[1];
            }
  #pragma unroll
            for (int nt = 0; nt < Dv / 8; ++nt) {
              o[rt][nt][0] *= corr[0]; o[rt][nt][1] *= corr[0]; o[rt][nt][2] *= corr[1]; o[rt][nt][3] *= corr[1];
            }
          }
        }
        // ---- value product on the codes, group by group: p * s_v as a two-term binary16 sum (high part + rounded
        // remainder) is the A operand, which keeps the product good to ~2^-22 whatever the cached magnitudes ----
        bool any_active = false;
  #pragma unroll
        for (int rt = 0; rt < R; ++rt) any_active |= active[rt];
        if (any_active) {
  #pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            uint32_t apv[R][2][4], apl[R][2][4];           // [tile][MMA][register]
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              float2 v[2];                                 // (scale, bias) of tokens e = 0, 1 for this group
              if (G == 2) {
                const uint4 sb = vsb4[i * 4 + tid];
                v[0] = sb_to_f2<kBf>(gi == 0 ? sb.x : sb.y); v[1] = sb_to_f2<kBf>(gi == 0 ? sb.z : sb.w);
              } else {
  #pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const uint4 sb = vsb4[(i * 4 + tid) * 2 + e];
                  v[e] = sb_to_f2<kBf>(gi == 0 ? sb.x : gi == 1 ? sb.y : gi == 2 ? sb.z : sb.w);
                }
              }
              if (tail) {
  #pragma unroll
                for (int e = 0; e < 2; ++e)
                  if (pos0 + 8 * tid + 4 * e + i >= kv_len) v[e] = make_float2(0.f, 0.f);
              }
  #pragma unroll
              for (int rt = 0; rt < R; ++rt) {
                if (!active[rt]) continue;
  #pragma unroll
                for (int r = 0; r < 2; ++r) {
                  const float x0 = prob[rt][i][0][r] * v[0].x, x1 = prob[rt][i][1][r] * v[1].x;
                  const uint32_t hi = f32x2_to_h2(x0, x1);
                  const float2 hf = h2_to_f2(hi);
                  apv[rt][i >> 1][(i & 1) * 2 + r] = hi;
                  apl[rt][i >> 1][(i & 1) * 2 + r] = f32x2_to_h2(x0 - hf.x, x1 - hf.y);
                  const float b = fmaf(prob[rt][i][0][r], v[0].y, prob[rt][i][1][r] * v[1].y);
                  if (i & 1) bias_o[rt][r][gi] += b; else bias_e[rt][r][gi] += b;
                }
              }
            }
  #pragma unroll
            for (int q4 = 2 * gi; q4 < 2 * gi + 2; ++q4) {
              const uint4 w4 = vc4[(q4 * 8 + g) * 4 + tid];
              const uint32_t wd[4] = {w4.x, w4.y, w4.z, w4.w};
  #pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint32_t wh = wd[j] >> 8;
                const uint32_t be0 = wd[j] & kMaskLo, be1 = wd[j] & kMaskHi, bo0 = wh & kMaskLo, bo1 = wh & kMaskHi;
  #pragma unroll
                for (int rt = 0; rt < R; ++rt) {
                  if (!active[rt]) continue;
                  mma_f16(o[rt][4 * q4 + j], apv[rt][0], be0, be1);
                  mma_f16(o[rt][4 * q4 + j], apv[rt][1], bo0, bo1);
                  mma_f16(o[rt][4 * q4 + j], apl[rt][0], be0, be1);
                  mma_f16(o[rt][4 * q4 + j], apl[rt][1], bo0, bo1);
                }
              }
            }
          }
        }
      }
    }
    // ---- release the slot; the warp that completes the count refills it ----
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      const int old = atomicAdd(&sm.released[slot], 1);
      if (old == kWarps * (round + 1) - 1 && k + kSlots < n_chunks) issue(k + kSlots);
    }
  }
  if (aborted && lane == 0) {
    raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
    // giving up: the copies already issued into the ring land before this warp lets go of shared memory.  Slot s has
    // received one copy per completed round of releases plus the first one.
    for (int s = 0; s < kSlots && s < n_chunks; ++s) {
      const int later = (n_chunks - 1 - s) / kSlots;                       // refills this slot can ever get
      const int issued = 1 + min(*(volatile int*)&sm.released[s] / kWarps, later);
      for (uint32_t i = 0; i < 4096u && !mbar_try_wait(&sm.full[s], (uint32_t)(issued - 1) & 1u); ++i) {}
    }
  }

  // ---- normalise and write this warp's rows ----
  if (h >= n_rep) return;
#pragma unroll
  for (int rt = 0; rt < R; ++rt)
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      float l = l_e[rt][r] + 16.f * l_o[rt][r];
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
      float bias[G];
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        float b = bias_e[rt][r][gi] + 16.f * bias_o[rt][r][gi];
        b += __shfl_xor_sync(0xffffffffu, b, 1);
        b += __shfl_xor_sync(0xffffffffu, b, 2);
        bias[gi] = b;
      }
      const int i = i_min + (qhalf * R + rt) * 16 + g + 8 * r;
      if (i >= q_len) continue;
      if (poisoned || aborted) l = 0.f;
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const size_t row = (size_t)(q0 + i) * y.Hq + (size_t)hk * n_rep + h;
#pragma unroll
      for (int nt = 0; nt < Dv / 8; ++nt) {
        const float v0 = (o[rt][nt][2 * r] * 16777216.f + bias[nt >> 3]) * inv;
        const float v1 = (o[rt][nt][2 * r + 1] * 16777216.f + bias[nt >> 3]) * inv;
        const int d = 8 * nt + 2 * tid;
        if (P.out_dtype == Q4KV_OUT_BF16) {
          *reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(P.out) + row * Dv + d) = __floats2bfloat162_rn(v0, v1);
        } else {
          *reinterpret_cast<float2*>(reinterpret_cast<float*>(P.out) + row * Dv + d) = make_float2(v0, v1);
        }
      }
      if (tid == 0 && P.lse) P.lse[row] = l > 0.f ? (m_run[rt][r] + log2f(l)) / kLog2e : -INFINITY;
    }
}

template <int R, int G, bool kBf>
cudaError_t launch_r(const PrefillParams& P, dim3 grid, cudaStream_t st) {
  static bool configured[64] = {};
  const size_t smem = sizeof(PrefillSmem<R, G>);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(prefill_mma_kernel<R, G, kBf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, prefill_mma_kernel<R, G, kBf>, P);
}

}  // namespace

bool prefill_mma_supported(const Layout& y) { return !y.alias && y.D == y.Dv && (y.D == 128 || y.D == 256) && y.n_rep <= 4; }

cudaError_t launch_prefill_mma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                               const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window, const void* q,
                               float scale, void* out, int out_dtype, float* lse, int32_t* flags, cudaStream_t st) {
  if (b.n_agents <= 0 || max_q_len <= 0) return cudaSuccess;
  PrefillParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.q_offs = q_offs; P.window = window;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e; P.out = out; P.out_dtype = out_dtype; P.lse = lse; P.flags = flags;
  const int hs = y.n_rep > 2 ? 4 : y.n_rep;
  const int tile1 = (kWarps / hs) * 16;                  // queries per CTA with one 16-row tile per warp
  if (y.G == 4) {
    // d = 256: one 16-row tile per warp (the accumulators of a tile are 128 registers per lane)
    const dim3 grid((max_q_len + tile1 - 1) / tile1, y.Hkv, b.n_agents);
    return y.sb_bf16 ? launch_r<1, 4, true>(P, grid, st) : launch_r<1, 4, false>(P, grid, st);
  }
  const dim3 grid((max_q_len + 2 * tile1 - 1) / (2 * tile1), y.Hkv, b.n_agents);
  return y.sb_bf16 ? launch_r<2, 2, true>(P, grid, st) : launch_r<2, 2, false>(P, grid, st);
}

}  // namespace q4kv
