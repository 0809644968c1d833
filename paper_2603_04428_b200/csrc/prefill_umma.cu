// q4kv_prefill_attention, tcgen05 path (d_qk = d_v = 128; 1, 2 or 4 query heads per KV head): the
// queries of a new phase over the cached Q4 prefix plus the causal new tokens, read from the Q4
// cache in place (Sections 3.4 "chunked prefill" and 3.5 "cross-phase context injection"; GQA and
// sliding windows: Section 3.6).
//
// Prefill is a dense contraction, so it runs on the fifth-generation tensor cores, and the 4-bit
// cache is expanded exactly once per CTA and key block, not once per query row:
//   * A CTA owns 256 score rows = two tiles of 128 rows (128 / n_rep consecutive queries x the n_rep
//     heads of one KV head) and walks the keys 64 at a time (two 32-token chunks, one bulk copy).
//   * Four "dequantize" warps turn each raw block into binary16 tiles K^ [64 keys][128 dims] and
//     V^ [128 dims][64 keys] in shared memory, in the core-matrix order a K-major tcgen05 operand
//     wants: x^ = c * s + b in one binary16 fma per pair of codes (the code is made a binary16
//     integer by or-ing the masked nibble into the mantissa of 1024 or 64 and subtracting), i.e.
//     each value is rounded once, to 11 significant bits.  A packed word becomes one 16-byte row of
//     a core matrix; the order of the eight elements inside a row (0,4,1,5,2,6,3,7) is absorbed by
//     storing the queries, and the key rows, in the same order.
//   * One thread issues the MMAs: S_t = Q_t K^T (M 128, N 64, K 128) with Q_t resident in tensor
//     memory as packed binary16 (each bf16 query row scaled by a power of two, so nothing is
//     rounded), and O_t += P_t V^ (M 128, N 128, K 64) with P_t read from tensor memory too; the
//     f32 accumulators S_t and O_t live in tensor memory (512 columns: O 2 x 128, S 2 x 64, Q 2 x 64;
//     P_t overlays S_t).  Only the B operands come from shared memory, which keeps the operand
//     traffic at half of the shared-memory bandwidth and leaves the rest to the dequantize warps.
//   * Sixteen softmax warps, two threads per score row (a tensor-memory lane; each takes 32 of the
//     64 scores): mask, online softmax with a lazily updated reference maximum (the accumulator is
//     rescaled only when the maximum has grown by more than 2^8), write P_t as packed binary16.
//     The two tiles alternate, so one tile's softmax overlaps the other tile's MMAs.
//   * One warp streams the raw blocks through a small ring with bulk asynchronous copies.
// All hand-offs are mbarriers; every wait is bounded and a wait that runs out raises
// Q4KV_FLAG_INTERNAL, drains the tensor pipe and frees the tensor memory before the CTA returns.
#include "q4kv_layout.cuh"
#include "tcgen05.cuh"

namespace q4kv {

namespace {

using namespace tc;

constexpr int kSoftmaxWarps = 16, kDequantWarps = 4;
constexpr int kMmaWarp = kSoftmaxWarps + kDequantWarps, kLoadWarp = kMmaWarp + 1;
constexpr int kThreads = (kLoadWarp + 1) * 32;           // 704
constexpr int kStages = 3;                               // K^ / V^ tiles in flight
constexpr int kRawSlots = 4;                             // raw 64-key blocks in flight
constexpr int kChunkBytes = 4608;                        // d = 128: [Kc 2048 | Ksb 256 | Vc 2048 | Vsb 256]
constexpr int kRawBytes = 2 * kChunkBytes;
constexpr int kTileBytes = 64 * 128 * 2;                 // one binary16 tile
constexpr uint32_t kColO = 0, kColS = 256, kColQ = 384;  // tensor-memory columns (+128 t, +64 t, +64 t)
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
  const uint16_t* q;          // bf16 [total_q][Hq][128]
  float scale_log2;
  void* out;
  int out_dtype;
  float* lse;
  int32_t* flags;
};

struct UmmaSmem {
  alignas(128) uint8_t khat[kStages][kTileBytes];        // [key 64][dim 128]: (n%8)*16 + (n/8)*2048 + (k/8)*128
  alignas(128) uint8_t vhat[kStages][kTileBytes];        // [dim 128][key 64]: (n%8)*16 + (n/8)*1024 + (k/8)*128
  alignas(128) uint8_t raw[kRawSlots][kRawBytes];
  alignas(8) uint64_t raw_full[kRawSlots], raw_free[kRawSlots], sb_done[kRawSlots];
  uint64_t k_full[kStages], v_full[kStages], kv_free[kStages];
  uint64_t s_full[2], p_full[2], o_done[2], q_ready, drain;
  uint32_t tmem_base;
  int bad[kRawSlots];
  float xchg[2][2][2][128];                              // [tile][parity][column half][row]: maxima / sums of the two threads of a row
  int stop[2][3], spoiled[2];
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

template <bool kBf>
__global__ void __launch_bounds__(kThreads, 1) prefill_umma_kernel(const __grid_constant__ UmmaParams P) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  UmmaSmem& sm = *reinterpret_cast<UmmaSmem*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = blockIdx.x, hk = blockIdx.y, a = blockIdx.z;
  const int n_rep = y.n_rep;
  const int tile_q = 128 / n_rep;                        // queries per 128-row tile

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- this CTA's queries and key range (inputs no kernel writes) ----
  const int q0 = P.q_offs[a], q_len = P.q_offs[a + 1] - q0;
  const int kv_len = P.kv_lens[a];
  const int i_min = qt * 2 * tile_q;
  if (i_min >= q_len) return;                            // uniform: nothing allocated, no barrier passed
  const bool bad_len = kv_len < 0 || kv_len > P.max_blocks * kBlockTokens || q_len > kv_len;
  const int i_max = min(q_len, i_min + 2 * tile_q) - 1;
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
      mbar_init(&sm.k_full[s], kDequantWarps); mbar_init(&sm.v_full[s], kDequantWarps); mbar_init(&sm.kv_free[s], 1);
    }
    for (int t = 0; t < 2; ++t) { mbar_init(&sm.s_full[t], 1); mbar_init(&sm.p_full[t], 256); mbar_init(&sm.o_done[t], 1); }
    mbar_init(&sm.q_ready, 512);
    for (int i = 0; i < 6; ++i) (&sm.stop[0][0])[i] = 0;
    sm.spoiled[0] = 0; sm.spoiled[1] = 0;
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
    const int x = threadIdx.x - kSoftmaxWarps * 32;      // 0..127
    // K: one 16-byte piece (words w = 4j + kt, j = 0..3) of token tau = 4 kg + ki per chunk.  The eight lanes
    // of a shared-memory phase read eight different 16-byte columns and write eight different rows.
    const int ki = x & 3, kg = 2 * ((x >> 3) & 3) + ((x >> 2) & 1), kt = (ki + (x >> 5)) & 3;
    const int ktau = 4 * kg + ki;
    const int k_read = (ki * 32 + kg * 4 + kt) * 16;
    const int k_sb = 2048 + (((ktau & 3) * 4 + (ktau >> 3)) * 2 + ((ktau >> 2) & 1)) * 8;
    const int k_row = 8 * (ktau >> 3) + slot_of(ktau & 7);       // row of the token inside its chunk's 32 rows
    // V: one 16-byte piece (dims 32 vq + 8 k + vr, k = 0..3) of token octet vo per chunk.
    const int vr = x & 7, vq = (x >> 3) & 3, vo = ((vr >> 1) + (x >> 5)) & 3;
    const int v_read = 2304 + ((vq * 8 + vr) * 4 + vo) * 16;
    const int v_sb = 4352 + (vo * 2 * 2 + (vq >> 1)) * 4;        // + i * 64 + e * 8: token 8 vo + 4 e + i, group vq / 2
    for (int j = 0; j < n_iter; ++j) {
      const int s = j % kStages, r = j % kRawSlots;
      if (j >= kStages && !mbar_wait(&sm.kv_free[s], (uint32_t)(j / kStages - 1), abort_flag)) break;
      if (!mbar_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots), abort_flag)) break;
      const bool bad = sm.bad[r] != 0;
      const int pos_base = (it0 + j) * 64;
      if (kBf) {
        // bfloat16 scales and biases become binary16 in place, once per block (the tiles are binary16); only the
        // tokens below the agent's length count for the range report (bytes past the end are whatever was there)
        bool overflow = false;
        for (int w = x; w < 256; w += kDequantWarps * 32) {              // per chunk: 64 words of Ksb, 64 of Vsb
          const int ci = w >> 7, o = w & 127;
          const int row = (o & 63) >> 1;                                 // (i * 4 + tid) * 2 + e: token 8 tid + 4 e + i
          const int tau = 8 * ((row >> 1) & 3) + 4 * (row & 1) + (row >> 3);
          uint32_t* at = reinterpret_cast<uint32_t*>(sm.raw[r] + ci * kChunkBytes + (o < 64 ? 2048 + 4 * o : 4352 + 4 * (o - 64)));
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
      for (int ci = 0; ci < 2; ++ci) {
        const uint8_t* chunk = sm.raw[r] + ci * kChunkBytes;
        const uint4 kw = *reinterpret_cast<const uint4*>(chunk + k_read);
        uint2 sb = *reinterpret_cast<const uint2*>(chunk + k_sb);          // (scale, bias) of groups 0 and 1
        if (bad || pos_base + ci * 32 + ktau >= kv_len) sb = make_uint2(0u, 0u);   // stale bytes past the end
        const uint32_t s0 = __byte_perm(sb.x, sb.x, 0x1010), b0 = __byte_perm(sb.x, sb.x, 0x3232);
        const uint32_t s1 = __byte_perm(sb.y, sb.y, 0x1010), b1 = __byte_perm(sb.y, sb.y, 0x3232);
        const int n = ci * 32 + k_row;
        uint8_t* dst = sm.khat[s] + (n & 7) * 16 + (n >> 3) * 2048 + kt * 128;
        *reinterpret_cast<uint4*>(dst + 0 * 512) = dequant8(kw.x, s0, b0, s0, b0, s0, b0, s0, b0);
        *reinterpret_cast<uint4*>(dst + 1 * 512) = dequant8(kw.y, s0, b0, s0, b0, s0, b0, s0, b0);
        *reinterpret_cast<uint4*>(dst + 2 * 512) = dequant8(kw.z, s1, b1, s1, b1, s1, b1, s1, b1);
        *reinterpret_cast<uint4*>(dst + 3 * 512) = dequant8(kw.w, s1, b1, s1, b1, s1, b1, s1, b1);
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.k_full[s]);
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const uint8_t* chunk = sm.raw[r] + ci * kChunkBytes;
        const uint4 vw = *reinterpret_cast<const uint4*>(chunk + v_read);
        uint32_t sp[4], bp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t e0 = *reinterpret_cast<const uint32_t*>(chunk + v_sb + i * 64);
          uint32_t e1 = *reinterpret_cast<const uint32_t*>(chunk + v_sb + i * 64 + 8);
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
      constexpr uint32_t kIdescS = idesc_f16(128, 64), kIdescO = idesc_f16(128, 128);
      auto issue_qk = [&](int t, int s) {                // S_t = Q_t K^T
        const uint32_t kb = smem_u32(sm.khat[s]);
#pragma unroll                                           // rolled, every MMA waits for its own operand arithmetic: 2x slower
        for (int k = 0; k < 8; ++k) {
          const uint64_t bd = smem_desc(kb + 256 * k, 128, 2048);
          if (elect_one()) mma_f16_ts(tb + kColS + 64 * t, tb + kColQ + 64 * t + 8 * k, bd, kIdescS, k > 0);
        }
        if (elect_one()) commit(&sm.s_full[t]);
      };
      auto issue_pv = [&](int t, int s, bool first) {    // O_t (+)= P_t V^
        const uint32_t vb = smem_u32(sm.vhat[s]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t bd = smem_desc(vb + 256 * k, 128, 1024);
          if (elect_one()) mma_f16_ts(tb + kColO + 128 * t, tb + kColS + 64 * t + 8 * k, bd, kIdescO, (!first || k > 0) ? 1u : 0u);
        }
        if (elect_one()) commit(&sm.o_done[t]);
      };
      bool ok = mbar_wait(&sm.q_ready, 0, abort_flag) && mbar_wait(&sm.k_full[0], 0, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        fence_after_sync();
        issue_qk(0, 0);
        issue_qk(1, 0);
      }
      for (int j = 0; ok && j < n_iter; ++j) {
        const int s = j % kStages, sn = (j + 1) % kStages;
        for (int t = 0; t < 2 && ok; ++t) {
          ok = mbar_wait(&sm.p_full[t], (uint32_t)j, abort_flag);
          if (ok && t == 0) ok = mbar_wait(&sm.v_full[s], (uint32_t)(j / kStages), abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          fence_after_sync();
          issue_pv(t, s, j == 0);
          if (t == 1 && elect_one()) commit(&sm.kv_free[s]);   // every MMA that reads stage s has been issued
          if (j + 1 < n_iter) {
            if (t == 0) ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[sn], (uint32_t)((j + 1) / kStages), abort_flag));
            if (!ok) break;
            fence_after_sync();
            issue_qk(t, sn);
          }
        }
      }
    }
  } else {
    // =============================== softmax warps: two threads per score row ===================
    // Warp w: tile t = w / 8, column half = (w / 4) % 2, tensor-memory lanes 32 (w % 4) ...  The two threads of a
    // row exchange their block maxima (and at the end their sums) through shared memory; the 256 threads of a
    // tile meet at a named barrier once per block, and they leave the loop together (one of them samples the
    // give-up flag before the barrier).
    const int t = warp >> 3, half = (warp >> 2) & 1;
    const int row = (warp & 3) * 32 + lane;              // tensor-memory lane
    const uint32_t lane_addr = tb + ((uint32_t)((warp & 3) * 32) << 16);
    const int h = row / tile_q, i = i_min + t * tile_q + row % tile_q;
    const bool valid = i < q_len && !bad_len;
    const int pq = prefix + i;                           // this row's position
    const bool sampler = (warp & 7) == 0 && lane == 0;   // one thread per tile
    auto tile_barrier = [&]() { asm volatile("bar.sync %0, 256;" ::"r"(1 + t) : "memory"); };
    float kappa;                                         // score in log2 units = S * kappa
    {
      // ---- stage this thread's half of the query row: bf16 -> binary16 times a power of two, element order
      //      (0,4,1,5,2,6,3,7) inside every eight ----
      const uint16_t* qrow = P.q + ((size_t)(q0 + (valid ? i : 0)) * y.Hq + (size_t)hk * n_rep + h) * 128 + 64 * half;
      uint32_t qa[32];
      float mx = 0.f;
      if (valid) {
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const uint4 v = *reinterpret_cast<const uint4*>(qrow + 8 * w);
          qa[4 * w] = v.x; qa[4 * w + 1] = v.y; qa[4 * w + 2] = v.z; qa[4 * w + 3] = v.w;
          mx = fmaxf(mx, fmaxf(fmaxf(fabsf(__uint_as_float(v.x << 16)), fabsf(__uint_as_float(v.x & 0xffff0000u))),
                               fmaxf(fabsf(__uint_as_float(v.y << 16)), fabsf(__uint_as_float(v.y & 0xffff0000u)))));
          mx = fmaxf(mx, fmaxf(fmaxf(fabsf(__uint_as_float(v.z << 16)), fabsf(__uint_as_float(v.z & 0xffff0000u))),
                               fmaxf(fabsf(__uint_as_float(v.w << 16)), fabsf(__uint_as_float(v.w & 0xffff0000u)))));
        }
      } else {
#pragma unroll
        for (int w = 0; w < 32; ++w) qa[w] = 0u;
      }
      sm.xchg[t][1][half][row] = mx;                     // slot 1: block 0 of the loop below writes slot 0
      tile_barrier();
      mx = fmaxf(mx, sm.xchg[t][1][half ^ 1][row]);
      int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
      if (mx == 0.f) ex = 0;
      ex = min(max(ex, -100), 100);
      const float sf = __uint_as_float((uint32_t)(127 + 8 - ex) << 23);      // 256 <= max |q| * sf < 512
      kappa = P.scale_log2 * __uint_as_float((uint32_t)(127 - 8 + ex) << 23);
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        // elements 8w..8w+7 arrive as bf16 pairs (0,1) (2,3) (4,5) (6,7); columns hold (0,4) (1,5) (2,6) (3,7)
        const uint32_t u01 = qa[4 * w], u23 = qa[4 * w + 1], u45 = qa[4 * w + 2], u67 = qa[4 * w + 3];
        const float x0 = __uint_as_float(u01 << 16) * sf, x1 = __uint_as_float(u01 & 0xffff0000u) * sf;
        const float x2 = __uint_as_float(u23 << 16) * sf, x3 = __uint_as_float(u23 & 0xffff0000u) * sf;
        const float x4 = __uint_as_float(u45 << 16) * sf, x5 = __uint_as_float(u45 & 0xffff0000u) * sf;
        const float x6 = __uint_as_float(u67 << 16) * sf, x7 = __uint_as_float(u67 & 0xffff0000u) * sf;
        qa[4 * w] = f32x2_to_h2(x0, x4); qa[4 * w + 1] = f32x2_to_h2(x1, x5);
        qa[4 * w + 2] = f32x2_to_h2(x2, x6); qa[4 * w + 3] = f32x2_to_h2(x3, x7);
      }
      tmem_st32(lane_addr + kColQ + 64 * t + 32 * half, qa);
      wait_st();
      fence_before_sync();
      mbar_arrive(&sm.q_ready);
    }
    float m_ref = -INFINITY, l = 0.f;                    // p = 2^(s - m_ref); m_ref trails the true maximum by at most kLazy
    for (int j = 0; j < n_iter; ++j) {
      mbar_wait(&sm.s_full[t], (uint32_t)j, abort_flag); // a wait that runs out raises the give-up flag; all leave below
      fence_after_sync();
      uint32_t sr[32];
      tmem_ld32(lane_addr + kColS + 64 * t + 32 * half, sr);
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
      sm.xchg[t][j & 1][half][row] = cm;
      if (sampler) sm.stop[t][j % 3] = *abort_flag;
      tile_barrier();                                    // also: every score of the tile has been read (P overlays S)
      if (sm.stop[t][j % 3]) break;
      cm = fmaxf(cm, sm.xchg[t][j & 1][half ^ 1][row]);
      if (cm != -INFINITY) cm *= kappa;                  // kappa > 0
      const float m_new = fmaxf(m_ref, cm);
      const bool grow = m_new > m_ref + kLazy || (m_ref == -INFINITY && m_new != -INFINITY);
      if (__any_sync(0xffffffffu, grow)) {
        if (j > 0) {
          // rescale this thread's half of the accumulator row: the previous block's value product must have landed
          mbar_wait(&sm.o_done[t], (uint32_t)(j - 1), abort_flag);
          fence_after_sync();
          const float f = grow ? fast_exp2(m_ref - m_new) : 1.f;           // m_ref = -inf: 0
#pragma unroll 1
          for (int part = 0; part < 2; ++part) {
            uint32_t orow[32];
            tmem_ld32(lane_addr + kColO + 128 * t + 64 * half + 32 * part, orow);
            wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) orow[c] = __float_as_uint(__uint_as_float(orow[c]) * f);
            tmem_st32(lane_addr + kColO + 128 * t + 64 * half + 32 * part, orow);
          }
          if (grow) l *= f;
        }
        if (grow) m_ref = m_new;
        probabilities(m_ref == -INFINITY ? 0.f : -m_ref);
      }
      l += sum;
      tmem_st16(lane_addr + kColS + 64 * t + 16 * half, pr);   // P_t overlays the first 32 columns of S_t
      wait_st();
      fence_before_sync();
      mbar_arrive(&sm.p_full[t]);
    }
    // ---- normalise and write this thread's half of the row ----
    bool ok = !*abort_flag;
    if (ok && n_iter > 0) ok = mbar_wait(&sm.o_done[t], (uint32_t)(n_iter - 1), abort_flag);
    const int slot = n_iter & 1;                         // not the slot the last block used
    sm.xchg[t][slot][half][row] = l;
    if (!ok) sm.spoiled[t] = 1;                          // anyone who gave up spoils the tile
    tile_barrier();
    ok = sm.spoiled[t] == 0;                             // uniform over the tile: the loads below are warp-wide
    l += sm.xchg[t][slot][half ^ 1][row];
    if (ok) fence_after_sync();
    const bool zero = !ok || n_iter == 0 || sm.poisoned != 0 || l <= 0.f;
    const float inv = zero ? 0.f : 1.f / l;
    const size_t orow_index = ((size_t)(q0 + i) * y.Hq + (size_t)hk * n_rep + h) * 128 + 64 * half;
#pragma unroll 1
    for (int part = 0; part < 2; ++part) {
      uint32_t orow[32];
      if (ok && n_iter > 0) {
        tmem_ld32(lane_addr + kColO + 128 * t + 64 * half + 32 * part, orow);
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
            const __nv_bfloat162 b = __floats2bfloat162_rn(zero ? 0.f : __uint_as_float(orow[c + 2 * e]) * inv,
                                                           zero ? 0.f : __uint_as_float(orow[c + 2 * e + 1]) * inv);
            vv[e] = *reinterpret_cast<const uint32_t*>(&b);
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

bool prefill_umma_supported(const Layout& y) {
  return !y.alias && y.D == 128 && y.Dv == 128 && (y.n_rep == 1 || y.n_rep == 2 || y.n_rep == 4);
}

cudaError_t launch_prefill_umma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                const int32_t* kv_lens, const int32_t* q_offs, int max_q_len, int window, const void* q,
                                float scale, void* out, int out_dtype, float* lse, int32_t* flags, cudaStream_t st) {
  if (b.n_agents <= 0 || max_q_len <= 0) return cudaSuccess;
  UmmaParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.q_offs = q_offs; P.window = window;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e; P.out = out; P.out_dtype = out_dtype; P.lse = lse; P.flags = flags;
  static bool configured[64][2] = {};
  const size_t smem = sizeof(UmmaSmem);
  const int bf = y.sb_bf16 ? 1 : 0;
  void (*kernel)(const UmmaParams) = bf ? prefill_umma_kernel<true> : prefill_umma_kernel<false>;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev][bf]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev][bf] = true;
  }
  const int cta_q = 2 * (128 / y.n_rep);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((max_q_len + cta_q - 1) / cta_q, y.Hkv, b.n_agents);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, P);
}

}  // namespace q4kv
