// q4kv_prefill_attention, tcgen05 path with one query tile per CTA, for the head shapes whose
// accumulator leaves no room for two: d_qk = d_v = 256 (the sliding-window model of Section 3.6) and
// d_qk 192 / d_v 128 (the per-head MLA cache of Section 3.6); 1, 2 or 4 query heads per KV head.  The
// queries of a new phase over the cached Q4 prefix plus the causal new tokens, read from the Q4
// cache in place (Sections 3.4 "chunked prefill" and 3.5 "cross-phase context injection").
//
// The d = 128 kernel's structure with one 128-row tile per CTA: at d = 256 a tile's accumulator
// alone is 256 of the 512 tensor-memory columns, and at 192 / 128 the queries of two tiles would not
// fit beside the accumulators.  What the second tile gave there -- its MMAs run while the first
// tile's softmax does -- comes here from two score buffers:
//   * A CTA owns 128 score rows (128 / n_rep consecutive queries x the n_rep heads of one KV head)
//     and walks the keys 64 at a time (two 32-token chunks, one bulk copy).
//   * Eight "dequantize" warps turn each raw block into binary16 tiles K^ [64 keys][d_qk] and
//     V^ [d_v][64 keys] in shared memory (two stages each), in the core-matrix order a K-major
//     tcgen05 operand wants: x^ = c * s + b in one binary16 fma per pair of codes, each value rounded
//     once to 11 significant bits.  A packed word becomes one 16-byte row of a core matrix; the order
//     of the eight elements inside a row (0,4,1,5,2,6,3,7) is absorbed by storing the queries, and
//     the key rows, in the same order.
//   * One thread issues the MMAs: S_b = Q K^T (M 128, N 64, K d_qk: d_qk / 16 instructions) into score
//     buffer b = block % 2, with Q resident in tensor memory as packed binary16 (each bf16 row scaled
//     by a power of two, so nothing is rounded), and O += P_b V^ (M 128, N d_v, K 64: 4 instructions)
//     with P_b read from tensor memory too, where it overlays S_b.  The scores of block j + 1 are
//     issued before the probabilities of block j exist, so the tensor pipe works through the softmax.
//     Tensor memory: O d_v columns, S 2 x 64, Q d_qk / 2.
//   * Eight softmax warps, two threads per score row (each takes 32 of the 64 scores and half of the
//     accumulator columns): mask, online softmax with a lazily updated reference maximum, P_b as
//     packed binary16.
//   * One warp streams the raw blocks through a three-slot ring with bulk asynchronous copies.
// All hand-offs are mbarriers; every wait is bounded and a wait that runs out raises
// Q4KV_FLAG_INTERNAL, drains the tensor pipe and frees the tensor memory before the CTA returns.
#include "q4kv_layout.cuh"
#include "tcgen05.cuh"

namespace q4kv {

namespace {

using namespace tc;

constexpr int kSoftmaxWarps = 8, kDequantWarps = 8;
constexpr int kMmaWarp = kSoftmaxWarps + kDequantWarps, kLoadWarp = kMmaWarp + 1;
constexpr int kThreads = (kLoadWarp + 1) * 32;           // 576
constexpr int kStages = 2;                               // K^ tiles, and V^ tiles, in flight
constexpr int kRawSlots = 3;                             // raw 64-key blocks in flight
constexpr uint32_t kColO = 0, kColS = 256, kColQ = 384;  // tensor-memory columns (d_v <= 256, 2 x 64, d_qk / 2 <= 128)
// G, Gv: groups of 64 along the key and value head dims
template <int G, int Gv>
struct Shape {
  static constexpr int D = 64 * G, Dv = 64 * Gv;
  static constexpr int kOffKsb = 16 * D, kOffVc = kOffKsb + 128 * G, kOffVsb = kOffVc + 16 * Dv;
  static constexpr int kChunkBytes = kOffVsb + 128 * Gv; // [Kc | Ksb | Vc | Vsb]: 9216 at 256 / 256, 5760 at 192 / 128
  static constexpr int kRawBytes = 2 * kChunkBytes;
  static constexpr int kTileK = 64 * D * 2, kTileV = Dv * 64 * 2;   // binary16 tiles
  static constexpr int kSboK = (D / 8) * 128;            // bytes between 8-key groups of K^
};
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLazy = 8.f;                             // rescale when the row maximum grew by more than this (log2)

struct UmmaParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks;
  const int32_t* tables;
  const int32_t* kv_lens;
  const int32_t* q_offs;
  int window;
  const uint16_t* q;          // bf16 [total_q][Hq][d_qk]
  float scale_log2;
  void* out;
  int out_dtype;
  float* lse;
  int32_t* flags;
};

template <int G, int Gv>
struct UmmaSmem {
  using Sh = Shape<G, Gv>;
  alignas(128) uint8_t khat[kStages][Sh::kTileK];        // [key 64][dim d_qk]: (n%8)*16 + (n/8)*kSboK + (k/8)*128
  alignas(128) uint8_t vhat[kStages][Sh::kTileV];        // [dim d_v][key 64]: (n%8)*16 + (n/8)*1024 + (k/8)*128
  alignas(128) uint8_t raw[kRawSlots][Sh::kRawBytes];
  alignas(8) uint64_t raw_full[kRawSlots], raw_free[kRawSlots], sb_done[kRawSlots];
  uint64_t k_full[kStages], v_full[kStages], k_free[kStages], v_free[kStages];
  uint64_t s_full[2], p_full[2], o_done, q_ready, drain;
  uint32_t tmem_base;
  int bad[kRawSlots];
  float xchg[2][2][128];                                 // [parity][column half][row]: maxima / sums of the two threads of a row
  int stop[3], spoiled;
  int abort_flag, poisoned;
};

// Eight codes of one packed word -> eight binary16 values c * s + b, as the pairs (0,4) (1,5) (2,6)
// (3,7) with the scale and bias pair given for each.  Masking a nibble into the mantissa of 1024
// (ulp 1) or of 64 (ulp 1/16, for a nibble sitting four bits up) gives 1024 + c or 64 + c exactly.
__device__ inline uint4 dequant8(uint32_t w, uint32_t s04, uint32_t b04, uint32_t s15, uint32_t b15, uint32_t s26,
                                 uint32_t b26, uint32_t s37, uint32_t b37) {
  const uint32_t wh = w >> 8;
  const __half2 k1024 = __half2half2(__ushort_as_half((unsigned short)0x6400));
  const __half2 k64 = __half2half2(__ushort_as_half((unsigned short)0x5400));
  auto as_h2 = [](uint32_t u) { return *reinterpret_cast<__half2*>(&u); };
  auto as_u = [](__half2 h) { return *reinterpret_cast<uint32_t*>(&h); };
  const __half2 c04 = __hsub2(as_h2((w & 0x000F000Fu) | 0x64006400u), k1024);
  const __half2 c15 = __hsub2(as_h2((w & 0x00F000F0u) | 0x54005400u), k64);
  const __half2 c26 = __hsub2(as_h2((wh & 0x000F000Fu) | 0x64006400u), k1024);
  const __half2 c37 = __hsub2(as_h2((wh & 0x00F000F0u) | 0x54005400u), k64);
  return make_uint4(as_u(__hfma2(c04, as_h2(s04), as_h2(b04))), as_u(__hfma2(c15, as_h2(s15), as_h2(b15))),
                    as_u(__hfma2(c26, as_h2(s26), as_h2(b26))), as_u(__hfma2(c37, as_h2(s37), as_h2(b37))));
}
// position inside a row's eight elements of element u (the inverse of 0,4,1,5,2,6,3,7)
__device__ inline int slot_of(int u) { return ((u & 3) << 1) | (u >> 2); }
// element held by slot j of a row
__device__ inline int elem_of(int j) { return ((j & 1) << 2) | (j >> 1); }
__device__ inline float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ inline uint32_t f32x2_to_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}
// A bfloat16 (scale, bias) pair as a binary16 pair: exact while the magnitude is a binary16 normal number (bfloat16
// has 8 significant bits), within 2^-25 below that; a magnitude beyond binary16's largest number is reported.
__device__ inline uint32_t bf16_pair_to_h2(uint32_t u, bool& overflow) {
  const uint32_t h = f32x2_to_h2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
  overflow |= (((h & 0x7C007C00u) + 0x04000400u) & 0x80008000u) != 0u;     // an exponent field of all ones
  return h;
}

template <int G, int Gv, bool kBf>
__global__ void __launch_bounds__(kThreads, 1) prefill_umma_1tile_kernel(const __grid_constant__ UmmaParams P) {
  using Sh = Shape<G, Gv>;
  constexpr int kD = Sh::D, kDv = Sh::Dv, kChunkBytes = Sh::kChunkBytes, kRawBytes = Sh::kRawBytes;
  constexpr int kOffKsb = Sh::kOffKsb, kOffVc = Sh::kOffVc, kOffVsb = Sh::kOffVsb;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  UmmaSmem<G, Gv>& sm = *reinterpret_cast<UmmaSmem<G, Gv>*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, hk = blockIdx.y, a = blockIdx.z;
  const int n_rep = y.n_rep;
  const int tile_q = 128 / n_rep;                        // queries of the CTA's 128-row tile

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- this CTA's queries and key range (inputs no kernel writes) ----
  const int q0 = P.q_offs[a], q_len = P.q_offs[a + 1] - q0;
  const int kv_len = P.kv_lens[a];
  const int i_min = qt * tile_q;
  if (i_min >= q_len) return;                            // uniform: nothing allocated, no barrier passed
  const bool bad_len = kv_len < 0 || kv_len > P.max_blocks * kBlockTokens || q_len > kv_len;
  const int i_max = min(q_len, i_min + tile_q) - 1;
  const int prefix = kv_len - q_len;                     // query i sits at position prefix + i
  const int W = P.window;
  const int c_end = bad_len ? 0 : (prefix + i_max) / 32 + 1;
  const int c_begin = (bad_len || W == 0) ? 0 : max(0, prefix + i_min - W + 1) >> 5;
  const int it0 = c_begin >> 1;                          // 64-key blocks it0 .. it0 + n_iter - 1
  const int n_iter = max(0, ((c_end + 1) >> 1) - it0);

  if (threadIdx.x == 0) {
    if (bad_len) raise_flag(P.flags, Q4KV_FLAG_BAD_LENGTH);
    for (int s = 0; s < kRawSlots; ++s) { mbar_init(&sm.raw_full[s], 1); mbar_init(&sm.raw_free[s], kDequantWarps); mbar_init(&sm.sb_done[s], kDequantWarps); sm.bad[s] = 0; }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.k_full[s], kDequantWarps); mbar_init(&sm.v_full[s], kDequantWarps);
      mbar_init(&sm.k_free[s], 1); mbar_init(&sm.v_free[s], 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm.s_full[b], 1); mbar_init(&sm.p_full[b], kSoftmaxWarps * 32); }
    mbar_init(&sm.o_done, 1);
    mbar_init(&sm.q_ready, kSoftmaxWarps * 32);
    for (int i = 0; i < 3; ++i) sm.stop[i] = 0;
    sm.spoiled = 0;
    mbar_init(&sm.drain, 1);
    sm.abort_flag = 0; sm.poisoned = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == kMmaWarp) { tmem_alloc(&sm.tmem_base, 512); tmem_relinquish(); }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tb = sm.tmem_base;
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the new tokens were appended by the preceding kernel
  volatile int* abort_flag = &sm.abort_flag;

  if (warp == kLoadWarp) {
    // =============================== raw block loader ==========================================
    if (lane == 0) {
      int issued = 0;
      for (int j = 0; j < n_iter; ++j) {
        const int r = j % kRawSlots;
        if (j >= kRawSlots && !mbar_wait(&sm.raw_free[r], (uint32_t)(j / kRawSlots - 1), abort_flag)) break;
        const int c = 2 * (it0 + j);
        const int blk = P.tables[(size_t)a * P.max_blocks + (c >> 3)];
        if (blk < 0 || blk >= P.n_blocks) {
          sm.bad[r] = 1;
          sm.poisoned = 1;
          raise_flag(P.flags, Q4KV_FLAG_BAD_BLOCK);
          mbar_arrive(&sm.raw_full[r]);
        } else {
          sm.bad[r] = 0;
          mbar_arrive_expect_tx(&sm.raw_full[r], kRawBytes);
          bulk_load(sm.raw[r], head_block(P.pool, y, P.layer, blk, hk) + (size_t)(c & 7) * kChunkBytes, kRawBytes,
                    &sm.raw_full[r]);
        }
        issued = j + 1;
      }
      // a CTA that is giving up still lets its own copies land before shared memory is released
      if (*abort_flag) {
        for (int j = max(0, issued - kRawSlots); j < issued; ++j) {
          const int r = j % kRawSlots;
          for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots) & 1u); ++i) {}
        }
      }
    }
  } else if (warp >= kSoftmaxWarps && warp < kMmaWarp) {
    // =============================== dequantize warps ==========================================
    // 256 threads.  At 256 / 256 a thread takes one of the two 16-byte key pieces of a token row (kj) and one value
    // piece, in both chunks of the block; at 192 / 128 a token row is a 16-byte and an 8-byte key piece and there are
    // half as many value pieces, and a thread works on one chunk of the block (c1).
    const int x = threadIdx.x - kSoftmaxWarps * 32;      // 0..255
    const int x7 = x & 127, c1 = x >> 7;
    // K: token tau = 4 kg + ki of a chunk, piece kt of its lane group.  The eight lanes of a shared-memory phase read
    // eight different 16-byte columns and write eight different rows.
    const int ki = x & 3, kg = 2 * ((x >> 3) & 3) + ((x >> 2) & 1), kt = (ki + (x7 >> 5)) & 3, kj = G == 4 ? c1 : 0;
    const int ktau = 4 * kg + ki;
    const int k_read = ki * (256 * G) + kj * 512 + kg * 64 + kt * 16;       // 16-byte piece: words 16 kj + kt + 4 m, m = 0..3
    const int k_read2 = ki * (256 * G) + 512 + kg * 32 + kt * 8;            // G = 3: the 8-byte piece, words 16 + kt, 20 + kt
    const int k_tok = ((ktau & 3) * 4 + (ktau >> 3)) * 2 + ((ktau >> 2) & 1);   // the token's place among the (scale, bias) rows
    const int k_sb = kOffKsb + (k_tok * G + 2 * kj) * 4;
    const int k_row = 8 * (ktau >> 3) + slot_of(ktau & 7);       // row of the token inside its chunk's 32 rows
    // V: one 16-byte piece (dims 32 vq + 8 k + vr, k = 0..3) of token octet vo per chunk.
    const int vr = x & 7, vq = ((x >> 3) & 3) + (Gv == 4 ? 4 * c1 : 0), vo = ((vr >> 1) + (x7 >> 5)) & 3;
    const int v_read = kOffVc + ((vq * 8 + vr) * 4 + vo) * 16;
    const int v_sb = kOffVsb + (vo * 2 * Gv + (vq >> 1)) * 4;    // + (i * 8 + e) * Gv * 4: token 8 vo + 4 e + i, group vq / 2
    constexpr int kChunksPerThread = G == 4 ? 2 : 1;
    for (int j = 0; j < n_iter; ++j) {
      const int s = j % kStages, r = j % kRawSlots;
      if (j >= kStages && !mbar_wait(&sm.k_free[s], (uint32_t)(j / kStages - 1), abort_flag)) break;
      if (!mbar_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots), abort_flag)) break;
      const bool bad = sm.bad[r] != 0;
      const int pos_base = (it0 + j) * 64;
      if (kBf) {
        // bfloat16 scales and biases become binary16 in place, once per block (the tiles are binary16); only the
        // tokens below the agent's length count for the range report (bytes past the end are whatever was there)
        constexpr int kSbWords = 32 * (G + Gv);          // per chunk: Ksb then Vsb
        bool overflow = false;
        for (int w = x; w < 2 * kSbWords; w += kDequantWarps * 32) {
          const int ci = w / kSbWords, o = w - ci * kSbWords;
          const bool is_k = o < 32 * G;
          const int row = is_k ? o / G : (o - 32 * G) / Gv;               // (i * 4 + tid) * 2 + e: token 8 tid + 4 e + i
          const int tau = 8 * ((row >> 1) & 3) + 4 * (row & 1) + (row >> 3);
          uint32_t* at = reinterpret_cast<uint32_t*>(sm.raw[r] + ci * kChunkBytes + (is_k ? kOffKsb + 4 * o : kOffVsb + 4 * (o - 32 * G)));
          bool over = false;
          *at = bf16_pair_to_h2(*at, over);
          overflow |= over && pos_base + ci * 32 + tau < kv_len;
        }
        if (overflow && !bad) raise_flag(P.flags, Q4KV_FLAG_SB_RANGE);
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.sb_done[r]);
        if (!mbar_wait(&sm.sb_done[r], (uint32_t)(j / kRawSlots), abort_flag)) break;
      }
#pragma unroll
      for (int cc = 0; cc < kChunksPerThread; ++cc) {
        const int ci = G == 4 ? cc : c1;
        const uint8_t* chunk = sm.raw[r] + ci * kChunkBytes;
        const bool dead = bad || pos_base + ci * 32 + ktau >= kv_len;      // stale bytes past the end
        const int n = ci * 32 + k_row;
        uint8_t* dst = sm.khat[s] + (n & 7) * 16 + (n >> 3) * Sh::kSboK + (16 * kj + kt) * 128;
        const uint4 kw = *reinterpret_cast<const uint4*>(chunk + k_read);
        uint32_t e0 = *reinterpret_cast<const uint32_t*>(chunk + k_sb);       // (scale, bias) of groups 2 kj and 2 kj + 1
        uint32_t e1 = *reinterpret_cast<const uint32_t*>(chunk + k_sb + 4);
        if (dead) { e0 = 0u; e1 = 0u; }
        const uint32_t s0 = __byte_perm(e0, e0, 0x1010), b0 = __byte_perm(e0, e0, 0x3232);
        const uint32_t s1 = __byte_perm(e1, e1, 0x1010), b1 = __byte_perm(e1, e1, 0x3232);
        *reinterpret_cast<uint4*>(dst + 0 * 512) = dequant8(kw.x, s0, b0, s0, b0, s0, b0, s0, b0);
        *reinterpret_cast<uint4*>(dst + 1 * 512) = dequant8(kw.y, s0, b0, s0, b0, s0, b0, s0, b0);
        *reinterpret_cast<uint4*>(dst + 2 * 512) = dequant8(kw.z, s1, b1, s1, b1, s1, b1, s1, b1);
        *reinterpret_cast<uint4*>(dst + 3 * 512) = dequant8(kw.w, s1, b1, s1, b1, s1, b1, s1, b1);
        if (G == 3) {
          const uint2 kw2 = *reinterpret_cast<const uint2*>(chunk + k_read2);
          uint32_t e2 = *reinterpret_cast<const uint32_t*>(chunk + k_sb + 8);  // group 2
          if (dead) e2 = 0u;
          const uint32_t s2 = __byte_perm(e2, e2, 0x1010), b2 = __byte_perm(e2, e2, 0x3232);
          *reinterpret_cast<uint4*>(dst + 4 * 512) = dequant8(kw2.x, s2, b2, s2, b2, s2, b2, s2, b2);
          *reinterpret_cast<uint4*>(dst + 5 * 512) = dequant8(kw2.y, s2, b2, s2, b2, s2, b2, s2, b2);
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.k_full[s]);
      if (j >= kStages && !mbar_wait(&sm.v_free[s], (uint32_t)(j / kStages - 1), abort_flag)) break;
#pragma unroll
      for (int cc = 0; cc < kChunksPerThread; ++cc) {
        const int ci = G == 4 ? cc : c1;
        const uint8_t* chunk = sm.raw[r] + ci * kChunkBytes;
        const uint4 vw = *reinterpret_cast<const uint4*>(chunk + v_read);
        uint32_t sp[4], bp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t e0 = *reinterpret_cast<const uint32_t*>(chunk + v_sb + i * 32 * Gv);
          uint32_t e1 = *reinterpret_cast<const uint32_t*>(chunk + v_sb + i * 32 * Gv + 4 * Gv);
          const int pos = pos_base + ci * 32 + 8 * vo + i;
          if (bad || pos >= kv_len) e0 = 0u;
          if (bad || pos + 4 >= kv_len) e1 = 0u;
          sp[i] = __byte_perm(e0, e1, 0x5410);                             // scales of tokens i and i + 4
          bp[i] = __byte_perm(e0, e1, 0x7632);                             // biases
        }
        uint8_t* dst = sm.vhat[s] + vr * 16 + (4 * vq) * 1024 + (ci * 4 + vo) * 128;
        *reinterpret_cast<uint4*>(dst + 0 * 1024) = dequant8(vw.x, sp[0], bp[0], sp[1], bp[1], sp[2], bp[2], sp[3], bp[3]);
        *reinterpret_cast<uint4*>(dst + 1 * 1024) = dequant8(vw.y, sp[0], bp[0], sp[1], bp[1], sp[2], bp[2], sp[3], bp[3]);
        *reinterpret_cast<uint4*>(dst + 2 * 1024) = dequant8(vw.z, sp[0], bp[0], sp[1], bp[1], sp[2], bp[2], sp[3], bp[3]);
        *reinterpret_cast<uint4*>(dst + 3 * 1024) = dequant8(vw.w, sp[0], bp[0], sp[1], bp[1], sp[2], bp[2], sp[3], bp[3]);
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&sm.v_full[s]); mbar_arrive(&sm.raw_free[r]); }
    }
  } else if (warp == kMmaWarp) {
    // =============================== MMA issue ==================================================
    // The whole warp runs this code, so that operands are computed once for the warp, and one elected
    // lane (always the same) issues the MMAs and the commits.
    if (n_iter > 0) {
      constexpr uint32_t kIdescS = idesc_f16(128, 64), kIdescO = idesc_f16(128, kDv);
      auto issue_qk = [&](int b, int s) {                // S_b = Q K^T; afterwards the K^ stage is free
        const uint32_t kb = smem_u32(sm.khat[s]);
#pragma unroll
        for (int k = 0; k < kD / 16; ++k) {
          const uint64_t bd = smem_desc(kb + 256 * k, 128, Sh::kSboK);
          if (elect_one()) mma_f16_ts(tb + kColS + 64 * b, tb + kColQ + 8 * k, bd, kIdescS, k > 0);
        }
        if (elect_one()) { commit(&sm.s_full[b]); commit(&sm.k_free[s]); }
      };
      auto issue_pv = [&](int b, int s, bool first) {    // O (+)= P_b V^; afterwards the V^ stage is free
        const uint32_t vb = smem_u32(sm.vhat[s]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t bd = smem_desc(vb + 256 * k, 128, 1024);
          if (elect_one()) mma_f16_ts(tb + kColO, tb + kColS + 64 * b + 8 * k, bd, kIdescO, (!first || k > 0) ? 1u : 0u);
        }
        if (elect_one()) { commit(&sm.o_done); commit(&sm.v_free[s]); }
      };
      bool ok = mbar_wait(&sm.q_ready, 0, abort_flag) && mbar_wait(&sm.k_full[0], 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        fence_after_sync();
        issue_qk(0, 0);
        if (n_iter > 1) {
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[1], 0, abort_flag));
          if (ok) {
            fence_after_sync();
            issue_qk(1, 1);
          }
        }
      }
      for (int j = 0; ok && j < n_iter; ++j) {
        const int b = j & 1, s = j % kStages;
        ok = mbar_wait(&sm.p_full[b], (uint32_t)(j >> 1), abort_flag) && mbar_wait(&sm.v_full[s], (uint32_t)(j / kStages), abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        fence_after_sync();
        issue_pv(b, s, j == 0);
        if (j + 2 < n_iter) {                            // the scores of block j + 2 replace P_b once the product above has read it
          ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[s], (uint32_t)((j + 2) / kStages), abort_flag));
          if (!ok) break;
          fence_after_sync();
          issue_qk(b, s);
        }
      }
    }
  } else {
    // =============================== softmax warps: two threads per score row ===================
    // Warp w: column half = w / 4, tensor-memory lanes 32 (w % 4) ...  The two threads of a row exchange their block
    // maxima (and at the end their sums) through shared memory; the 256 threads meet at a named barrier once per
    // block, and they leave the loop together (one of them samples the give-up flag before the barrier).
    const int half = (warp >> 2) & 1;
    const int row = (warp & 3) * 32 + lane;              // tensor-memory lane
    const uint32_t lane_addr = tb + ((uint32_t)((warp & 3) * 32) << 16);
    const int h = row / tile_q, i = i_min + row % tile_q;
    const bool valid = i < q_len && !bad_len;
    const int pq = prefix + i;                           // this row's position
    const bool sampler = warp == 0 && lane == 0;
    auto tile_barrier = [&]() { asm volatile("bar.sync 1, 256;" ::: "memory"); };
    float kappa;                                         // score in log2 units = S * kappa
    {
      // ---- stage this thread's half of the query row: bf16 -> binary16 times a power of two, element order
      //      (0,4,1,5,2,6,3,7) inside every eight ----
      constexpr int kQWords = kD / 4;                    // packed binary16 words of this thread's half row: 64 or 48
      const uint16_t* qrow = P.q + ((size_t)(q0 + (valid ? i : 0)) * y.Hq + (size_t)hk * n_rep + h) * kD + (kD / 2) * half;
      uint32_t qa[kQWords];
      float mx = 0.f;
      if (valid) {
#pragma unroll
        for (int w = 0; w < kQWords / 4; ++w) {
          const uint4 v = *reinterpret_cast<const uint4*>(qrow + 8 * w);
          qa[4 * w] = v.x; qa[4 * w + 1] = v.y; qa[4 * w + 2] = v.z; qa[4 * w + 3] = v.w;
          mx = fmaxf(mx, fmaxf(fmaxf(fabsf(__uint_as_float(v.x << 16)), fabsf(__uint_as_float(v.x & 0xffff0000u))),
                               fmaxf(fabsf(__uint_as_float(v.y << 16)), fabsf(__uint_as_float(v.y & 0xffff0000u)))));
          mx = fmaxf(mx, fmaxf(fmaxf(fabsf(__uint_as_float(v.z << 16)), fabsf(__uint_as_float(v.z & 0xffff0000u))),
                               fmaxf(fabsf(__uint_as_float(v.w << 16)), fabsf(__uint_as_float(v.w & 0xffff0000u)))));
        }
      } else {
#pragma unroll
        for (int w = 0; w < kQWords; ++w) qa[w] = 0u;
      }
      sm.xchg[1][half][row] = mx;                        // slot 1: block 0 of the loop below writes slot 0
      tile_barrier();
      mx = fmaxf(mx, sm.xchg[1][half ^ 1][row]);
      int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
      if (mx == 0.f) ex = 0;
      ex = min(max(ex, -100), 100);
      const float sf = __uint_as_float((uint32_t)(127 + 8 - ex) << 23);      // 256 <= max |q| * sf < 512
      kappa = P.scale_log2 * __uint_as_float((uint32_t)(127 - 8 + ex) << 23);
#pragma unroll
      for (int w = 0; w < kQWords / 4; ++w) {
        // elements 8w..8w+7 arrive as bf16 pairs (0,1) (2,3) (4,5) (6,7); columns hold (0,4) (1,5) (2,6) (3,7)
        const uint32_t u01 = qa[4 * w], u23 = qa[4 * w + 1], u45 = qa[4 * w + 2], u67 = qa[4 * w + 3];
        const float x0 = __uint_as_float(u01 << 16) * sf, x1 = __uint_as_float(u01 & 0xffff0000u) * sf;
        const float x2 = __uint_as_float(u23 << 16) * sf, x3 = __uint_as_float(u23 & 0xffff0000u) * sf;
        const float x4 = __uint_as_float(u45 << 16) * sf, x5 = __uint_as_float(u45 & 0xffff0000u) * sf;
        const float x6 = __uint_as_float(u67 << 16) * sf, x7 = __uint_as_float(u67 & 0xffff0000u) * sf;
        qa[4 * w] = f32x2_to_h2(x0, x4); qa[4 * w + 1] = f32x2_to_h2(x1, x5);
        qa[4 * w + 2] = f32x2_to_h2(x2, x6); qa[4 * w + 3] = f32x2_to_h2(x3, x7);
      }
      // 32-column stores start at multiples of 32 columns, 16-column stores at multiples of 16
      if (kQWords == 64) {
        tmem_st32(lane_addr + kColQ + 64 * half, qa);
        tmem_st32(lane_addr + kColQ + 64 * half + 32, qa + 32);
      } else if (half == 0) {
        tmem_st32(lane_addr + kColQ, qa);
        tmem_st16(lane_addr + kColQ + 32, qa + 32);
      } else {
        tmem_st16(lane_addr + kColQ + 48, qa);
        tmem_st32(lane_addr + kColQ + 64, qa + 16);
      }
      wait_st();
      fence_before_sync();
      mbar_arrive(&sm.q_ready);
    }
    float m_ref = -INFINITY, l = 0.f;                    // p = 2^(s - m_ref); m_ref trails the true maximum by at most kLazy
    for (int j = 0; j < n_iter; ++j) {
      const int b = j & 1;
      mbar_wait(&sm.s_full[b], (uint32_t)(j >> 1), abort_flag);   // a wait that runs out raises the give-up flag; all leave below
      fence_after_sync();
      uint32_t sr[32];
      tmem_ld32(lane_addr + kColS + 64 * b + 32 * half, sr);
      wait_ld();
      const int pos0 = (it0 + j) * 64 + 32 * half;
      // column c of this half is key pos0 + (c & ~7) + elem_of(c & 7); causal and window masks on edge blocks only
      if (pos0 + 31 > pq || (W > 0 && pos0 <= pq - W)) {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int pos = pos0 + (c & ~7) + elem_of(c & 7);
          if (pos > pq || (W > 0 && pos <= pq - W)) sr[c] = 0xff800000u;   // -inf
        }
      }
      // Probabilities against the current reference, and the block maximum beside them (independent instruction
      // streams); only when some row's maximum has outgrown its reference is the reference moved, the accumulator
      // rescaled and the probabilities taken again.  The scores stay in registers meanwhile.
      float sum = 0.f;
      uint32_t pr[16];
      auto probabilities = [&](float neg_m) {
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int c = 0; c < 16; c += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sr[2 * c]), kappa, neg_m));
          const float p1 = fast_exp2(fmaf(__uint_as_float(sr[2 * c + 1]), kappa, neg_m));
          const float p2 = fast_exp2(fmaf(__uint_as_float(sr[2 * c + 2]), kappa, neg_m));
          const float p3 = fast_exp2(fmaf(__uint_as_float(sr[2 * c + 3]), kappa, neg_m));
          s0 += p0; s1 += p1; s2 += p2; s3 += p3;
          pr[c] = f32x2_to_h2(p0, p1);
          pr[c + 1] = f32x2_to_h2(p2, p3);
        }
        sum = (s0 + s1) + (s2 + s3);
      };
      probabilities(m_ref == -INFINITY ? 0.f : -m_ref);
      float cm4[4] = {__uint_as_float(sr[0]), __uint_as_float(sr[1]), __uint_as_float(sr[2]), __uint_as_float(sr[3])};
#pragma unroll
      for (int c = 4; c < 32; ++c) cm4[c & 3] = fmaxf(cm4[c & 3], __uint_as_float(sr[c]));
      float cm = fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3]));
      sm.xchg[j & 1][half][row] = cm;
      if (sampler) sm.stop[j % 3] = *abort_flag;
      tile_barrier();                                    // also: every score of the block has been read (P overlays S)
      if (sm.stop[j % 3]) break;
      cm = fmaxf(cm, sm.xchg[j & 1][half ^ 1][row]);
      if (cm != -INFINITY) cm *= kappa;                  // kappa > 0
      const float m_new = fmaxf(m_ref, cm);
      const bool grow = m_new > m_ref + kLazy || (m_ref == -INFINITY && m_new != -INFINITY);
      if (__any_sync(0xffffffffu, grow)) {
        if (j > 0) {
          // rescale this thread's half of the accumulator row: the previous block's value product must have landed
          mbar_wait(&sm.o_done, (uint32_t)(j - 1), abort_flag);
          fence_after_sync();
          const float f = grow ? fast_exp2(m_ref - m_new) : 1.f;           // m_ref = -inf: 0
#pragma unroll 1
          for (int part = 0; part < kDv / 64; ++part) {
            uint32_t orow[32];
            tmem_ld32(lane_addr + kColO + (kDv / 2) * half + 32 * part, orow);
            wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) orow[c] = __float_as_uint(__uint_as_float(orow[c]) * f);
            tmem_st32(lane_addr + kColO + (kDv / 2) * half + 32 * part, orow);
          }
          if (grow) l *= f;
        }
        if (grow) m_ref = m_new;
        probabilities(m_ref == -INFINITY ? 0.f : -m_ref);
      }
      l += sum;
      tmem_st16(lane_addr + kColS + 64 * b + 16 * half, pr);   // P_b overlays the first 32 columns of S_b
      wait_st();
      fence_before_sync();
      mbar_arrive(&sm.p_full[b]);
    }
    // ---- normalise and write this thread's half of the row ----
    bool ok = !*abort_flag;
    if (ok && n_iter > 0) ok = mbar_wait(&sm.o_done, (uint32_t)(n_iter - 1), abort_flag);
    const int slot = n_iter & 1;                         // not the slot the last block used
    sm.xchg[slot][half][row] = l;
    if (!ok) sm.spoiled = 1;                             // anyone who gave up spoils the tile
    tile_barrier();
    ok = sm.spoiled == 0;                                // uniform over the tile: the loads below are warp-wide
    l += sm.xchg[slot][half ^ 1][row];
    if (ok) fence_after_sync();
    const bool zero = !ok || n_iter == 0 || sm.poisoned != 0 || l <= 0.f;
    const float inv = zero ? 0.f : 1.f / l;
    const size_t orow_index = ((size_t)(q0 + i) * y.Hq + (size_t)hk * n_rep + h) * kDv + (kDv / 2) * half;
#pragma unroll 1
    for (int part = 0; part < kDv / 64; ++part) {
      uint32_t orow[32];
      if (ok && n_iter > 0) {
        tmem_ld32(lane_addr + kColO + (kDv / 2) * half + 32 * part, orow);
        wait_ld();
      }
      if (i >= q_len) continue;
      if (P.out_dtype == Q4KV_OUT_BF16) {
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(P.out) + orow_index + 32 * part;
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 v;
          uint32_t* vv = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 bb = __floats2bfloat162_rn(zero ? 0.f : __uint_as_float(orow[c + 2 * e]) * inv,
                                                            zero ? 0.f : __uint_as_float(orow[c + 2 * e + 1]) * inv);
            vv[e] = *reinterpret_cast<const uint32_t*>(&bb);
          }
          *reinterpret_cast<uint4*>(o + c) = v;
        }
      } else {
        float* o = reinterpret_cast<float*>(P.out) + orow_index + 32 * part;
#pragma unroll
        for (int c = 0; c < 32; c += 4)
          *reinterpret_cast<float4*>(o + c) =
              zero ? make_float4(0.f, 0.f, 0.f, 0.f)
                   : make_float4(__uint_as_float(orow[c]) * inv, __uint_as_float(orow[c + 1]) * inv,
                                 __uint_as_float(orow[c + 2]) * inv, __uint_as_float(orow[c + 3]) * inv);
      }
    }
    if (half == 0 && i < q_len && P.lse)
      P.lse[(size_t)(q0 + i) * y.Hq + (size_t)hk * n_rep + h] = zero ? -INFINITY : (m_ref + log2f(l)) / kLog2e;
  }

  // ---- teardown: nothing may be in flight in the tensor pipe when the columns are given back ----
  fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    if (sm.abort_flag) {
      if (elect_one()) {                                 // the lane that issued the MMAs
        commit(&sm.drain);
        for (uint32_t k = 0; k < kSpinLimit && !mbar_try_wait(&sm.drain, 0); ++k) {}
        raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
      }
      __syncwarp();
    }
    fence_after_sync();
    tmem_dealloc(tb, 512);
  }
}

}  // namespace

bool prefill_umma_1tile_supported(const Layout& y) {
  const bool shape = (y.D == 256 && y.Dv == 256) || (y.D == 192 && y.Dv == 128);
  return !y.alias && shape && (y.n_rep == 1 || y.n_rep == 2 || y.n_rep == 4);
}

namespace {
template <int G, int Gv, bool kBf>
cudaError_t launch_shape(const UmmaParams& P, int max_q_len, cudaStream_t st) {
  static bool configured[64] = {};
  const size_t smem = sizeof(UmmaSmem<G, Gv>);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(prefill_umma_1tile_kernel<G, Gv, kBf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const int cta_q = 128 / P.y.n_rep;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((max_q_len + cta_q - 1) / cta_q, P.y.Hkv, P.n_agents);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, prefill_umma_1tile_kernel<G, Gv, kBf>, P);
}
}  // namespace

cudaError_t launch_prefill_umma_1tile(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                      const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window,
                                      const void* q, float scale, void* out, int out_dtype, float* lse, int32_t* flags,
                                      cudaStream_t st) {
  if (b.n_agents <= 0 || max_q_len <= 0) return cudaSuccess;
  UmmaParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.q_offs = q_offs; P.window = window;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e; P.out = out; P.out_dtype = out_dtype; P.lse = lse; P.flags = flags;
  if (y.D == 256) return y.sb_bf16 ? launch_shape<4, 4, true>(P, max_q_len, st) : launch_shape<4, 4, false>(P, max_q_len, st);
  return y.sb_bf16 ? launch_shape<3, 2, true>(P, max_q_len, st) : launch_shape<3, 2, false>(P, max_q_len, st);
}

}  // namespace q4kv
