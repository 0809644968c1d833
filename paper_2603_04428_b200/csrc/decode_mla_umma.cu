// q4kv_decode_attention, tcgen05 path for the MLA-latent cache (d_qk = 576 = 512 latent + 64 rope,
// d_v = 512, V aliases the first 512 dims of K, one shared KV head, up to 16 query heads): one
// query token per agent in absorbed form over the Q4 latent cache, read in place (Section 3.4
// "Batched Quantized Inference"; the MLA cache of Section 3.6).
//
// Every key serves all 16 heads and is both key and value, so the cache bytes are expanded once
// into a binary16 tile and the tensor cores see it twice:
//   * Work is split along the keys: CTA (split, agent) walks its share of the agent's keys 64 at a
//     time (two 32-token chunks = one bulk copy of 20736 bytes), leaves an (acc, m, l) record per
//     head, and a small second kernel combines the records of an agent.
//   * Four dequantize warps turn each raw block into the tile K^ [64 keys][576 dims] in shared
//     memory (x^ = c * s + b, one binary16 fma per pair of codes, rounded once), in 8 x 16-byte
//     core matrices: read along the dims it is a K-major operand, read along the keys an MN-major one.
//   * One thread issues the MMAs with the keys on the M side, so that no tensor work is spent on
//     padding the 16 heads to 128 rows:
//         S^T [64 keys][16 heads]  = K^ (A, K-major)  x  Q (B: [16 heads][576 dims] binary16, K-major)
//         O^T [512 dims][16 heads] += K^ (A, MN-major, first 512 dims) x P^T (B, MN-major)
//     with f32 accumulators in tensor memory (S^T double-buffered, O^T as four 128-lane tiles).
//   * Four softmax warps: a thread owns one key (a tensor-memory lane of S^T) and its 16 scores.
//     The reference maximum of each head is shared by the CTA and updated lazily: a block whose
//     scores exceed it by more than 2^8 triggers an exact per-head maximum (shuffles + shared
//     memory) and a rescale of O^T; otherwise a block costs 16 exponentials per key and one
//     32-byte row of P^T.  Row sums stay per-thread until the end.
// Every wait is bounded (Q4KV_FLAG_INTERNAL when one runs out); the tensor pipe is drained and the
// tensor memory freed before the CTA returns.
#include "q4kv_layout.cuh"
#include "tcgen05.cuh"

namespace q4kv {

namespace {

using namespace tc;

constexpr int kD = 576, kDv = 512, kHeads = 16;
constexpr int kSoftmaxWarps = 4, kDequantWarps = 4;
constexpr int kMmaWarp = kSoftmaxWarps + kDequantWarps, kLoadWarp = kMmaWarp + 1;
constexpr int kThreads = (kLoadWarp + 1) * 32;           // 320
constexpr int kChunkBytes = 32 * (kD / 2 + 4 * (kD / 64));   // 10368: [Kc 9216 | Ksb 1152]
constexpr int kRawBytes = 2 * kChunkBytes;               // one 64-key block
constexpr int kTileBytes = 64 * kD * 2;                  // 73728
constexpr int kGroupStride = (kD / 8) * 128;             // 9216: bytes between 8-row groups of a [rows][576] tile
constexpr int kStages = 2, kRawSlots = 2;
constexpr uint32_t kColS = 0, kColO = 32;                // tensor-memory columns: S^T 2 x 16, O^T 4 x 16
constexpr uint32_t kTmemCols = 128;
constexpr int kRecStride = kDv + 2;                      // acc[512], m, l
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLazy = 8.f;

struct MlaParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks;
  const int32_t* tables;
  const int32_t* kv_lens;
  int window;
  const uint16_t* q;          // bf16 [n_agents][Hq][576]
  float scale_log2;
  int n_splits, blocks_per_split;
  float* records;             // [n_agents][n_splits][16][kRecStride]
  int32_t* flags;
};

struct MlaSmem {
  alignas(128) uint8_t khat[kStages][kTileBytes];        // [key 64][dim 576]: (key%8)*16 + (key/8)*9216 + (dim/8)*128
  alignas(128) uint8_t raw[kRawSlots][kRawBytes];
  alignas(128) uint8_t qtile[kHeads * kD * 2];           // [head 16][dim 576], same form
  alignas(128) uint8_t ptile[kHeads * 64 * 2];           // P^T: (key%8)*16 + (key/8)*128 + (head/8)*1024 + (head%8)*2
  float kappa[kHeads];                                   // score in log2 units = S * kappa[head]
  float wmax[kSoftmaxWarps][kHeads];
  float wsum[kSoftmaxWarps][kHeads];
  alignas(8) uint64_t raw_full[kRawSlots], raw_free[kRawSlots];
  uint64_t k_full[kStages], kv_free[kStages];
  uint64_t s_full[2], p_full, o_done, q_ready, drain;
  uint32_t tmem_base;
  int grow[3], stop[3];
  int bad[kRawSlots];
  int abort_flag, poisoned;
};

// Eight codes of one packed word -> eight binary16 values c * s + b in the order (0,4) (1,5) (2,6) (3,7),
// one (scale, bias) for all (s2 = (s, s), b2 = (b, b)).  Or-ing a masked nibble into the mantissa of 1024
// (ulp 1), or of 64 for a nibble four bits up (ulp 1/16), gives 1024 + c or 64 + c exactly.
__device__ inline uint4 dequant8(uint32_t w, uint32_t s2, uint32_t b2) {
  const uint32_t wh = w >> 8;
  const __half2 k1024 = __half2half2(__ushort_as_half((unsigned short)0x6400));
  const __half2 k64 = __half2half2(__ushort_as_half((unsigned short)0x5400));
  auto as_h2 = [](uint32_t u) { return *reinterpret_cast<__half2*>(&u); };
  auto as_u = [](__half2 h) { return *reinterpret_cast<uint32_t*>(&h); };
  const __half2 s = as_h2(s2), b = as_h2(b2);
  const __half2 c04 = __hsub2(as_h2((w & 0x000F000Fu) | 0x64006400u), k1024);
  const __half2 c15 = __hsub2(as_h2((w & 0x00F000F0u) | 0x54005400u), k64);
  const __half2 c26 = __hsub2(as_h2((wh & 0x000F000Fu) | 0x64006400u), k1024);
  const __half2 c37 = __hsub2(as_h2((wh & 0x00F000F0u) | 0x54005400u), k64);
  return make_uint4(as_u(__hfma2(c04, s, b)), as_u(__hfma2(c15, s, b)), as_u(__hfma2(c26, s, b)), as_u(__hfma2(c37, s, b)));
}
// element held by slot j of a 16-byte row
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
__device__ inline void softmax_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }   // the four softmax warps

__global__ void __launch_bounds__(kThreads, 1) decode_mla_kernel(const __grid_constant__ MlaParams P) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  MlaSmem& sm = *reinterpret_cast<MlaSmem*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, a = blockIdx.y;
  const int n_rep = y.Hq;                                // one KV head

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- this CTA's share of the agent's keys (inputs no kernel writes) ----
  int n = P.kv_lens[a];
  const bool bad_len = n < 0 || n > P.max_blocks * kBlockTokens;
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
    for (int s = 0; s < kRawSlots; ++s) { mbar_init(&sm.raw_full[s], 1); mbar_init(&sm.raw_free[s], kDequantWarps); sm.bad[s] = 0; }
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.k_full[s], kDequantWarps); mbar_init(&sm.kv_free[s], 1); }
    mbar_init(&sm.s_full[0], 1); mbar_init(&sm.s_full[1], 1);
    mbar_init(&sm.p_full, 128); mbar_init(&sm.o_done, 1); mbar_init(&sm.q_ready, 128); mbar_init(&sm.drain, 1);
    sm.grow[0] = 0; sm.grow[1] = 0; sm.grow[2] = 0;
    sm.stop[0] = 0; sm.stop[1] = 0; sm.stop[2] = 0;
    sm.abort_flag = 0; sm.poisoned = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == kMmaWarp) { tmem_alloc(&sm.tmem_base, kTmemCols); tmem_relinquish(); }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tb = sm.tmem_base;
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the new token was appended by the preceding kernel
  volatile int* abort_flag = &sm.abort_flag;

  if (warp == kLoadWarp) {
    // =============================== raw block loader ==========================================
    if (lane == 0) {
      int issued = 0;
      for (int j = 0; j < n_iter; ++j) {
        const int r = j % kRawSlots;
        if (j >= kRawSlots && !mbar_wait(&sm.raw_free[r], (uint32_t)(j / kRawSlots - 1), abort_flag)) break;
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
          bulk_load(sm.raw[r], head_block(P.pool, y, P.layer, blk, 0) + (size_t)(c & 7) * kChunkBytes, kRawBytes,
                    &sm.raw_full[r]);
        }
        issued = j + 1;
      }
      if (*abort_flag) {                                 // giving up: let this thread's copies land first
        for (int j = max(0, issued - kRawSlots); j < issued; ++j) {
          const int r = j % kRawSlots;
          for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots) & 1u); ++i) {}
        }
      }
    }
  } else if (warp >= kSoftmaxWarps && warp < kMmaWarp) {
    // =============================== dequantize warps ==========================================
    // Per chunk a thread owns token tau = 4 kg + ki and, of its 72 words, those with w % 4 == kt: four 16-byte
    // pieces (words p = 4j..4j+3, w = 4p + kt) and one 8-byte piece (p = 16, 17).  The eight lanes of a
    // shared-memory phase read eight different 16-byte columns and write eight different rows.
    const int x = threadIdx.x - kSoftmaxWarps * 32;
    const int ki = x & 3, kg = 2 * ((x >> 3) & 3) + ((x >> 2) & 1), kt = (ki + (x >> 5)) & 3;
    const int tau = 4 * kg + ki;
    const int rd16 = (ki * 144 + kg * 4 + kt) * 16;      // + j * 512
    const int rd8 = (ki * 576 + 512) * 4 + (kg * 4 + kt) * 8;
    const int sb_at = 9216 + ((((tau & 3) * 4 + (tau >> 3)) * 2 + ((tau >> 2) & 1)) * 9) * 4;   // + 4 * group
    for (int j = 0; j < n_iter; ++j) {
      const int s = j % kStages, r = j % kRawSlots;
      if (j >= kStages && !mbar_wait(&sm.kv_free[s], (uint32_t)(j / kStages - 1), abort_flag)) break;
      if (!mbar_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots), abort_flag)) break;
      const bool bad = sm.bad[r] != 0;
      const int pos_base = (b0 + j) * 64;
#pragma unroll 1
      for (int ci = 0; ci < 2; ++ci) {
        const uint8_t* chunk = sm.raw[r] + ci * kChunkBytes;
        const bool dead = bad || pos_base + ci * 32 + tau >= n;            // stale bytes past the end
        const int row = ci * 32 + tau;
        uint8_t* dst = sm.khat[s] + (row & 7) * 16 + (row >> 3) * kGroupStride + kt * 128;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const uint4 kw = *reinterpret_cast<const uint4*>(chunk + rd16 + jj * 512);
          uint32_t sb0 = *reinterpret_cast<const uint32_t*>(chunk + sb_at + 8 * jj);        // group 2 jj
          uint32_t sb1 = *reinterpret_cast<const uint32_t*>(chunk + sb_at + 8 * jj + 4);    // group 2 jj + 1
          if (dead) { sb0 = 0u; sb1 = 0u; }
          const uint32_t s0 = __byte_perm(sb0, sb0, 0x1010), c0 = __byte_perm(sb0, sb0, 0x3232);
          const uint32_t s1 = __byte_perm(sb1, sb1, 0x1010), c1 = __byte_perm(sb1, sb1, 0x3232);
          *reinterpret_cast<uint4*>(dst + (16 * jj + 0) * 128) = dequant8(kw.x, s0, c0);
          *reinterpret_cast<uint4*>(dst + (16 * jj + 4) * 128) = dequant8(kw.y, s0, c0);
          *reinterpret_cast<uint4*>(dst + (16 * jj + 8) * 128) = dequant8(kw.z, s1, c1);
          *reinterpret_cast<uint4*>(dst + (16 * jj + 12) * 128) = dequant8(kw.w, s1, c1);
        }
        {
          const uint2 kw = *reinterpret_cast<const uint2*>(chunk + rd8);
          uint32_t sb8 = *reinterpret_cast<const uint32_t*>(chunk + sb_at + 32);            // group 8
          if (dead) sb8 = 0u;
          const uint32_t s8 = __byte_perm(sb8, sb8, 0x1010), c8 = __byte_perm(sb8, sb8, 0x3232);
          *reinterpret_cast<uint4*>(dst + 64 * 128) = dequant8(kw.x, s8, c8);
          *reinterpret_cast<uint4*>(dst + 68 * 128) = dequant8(kw.y, s8, c8);
        }
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&sm.k_full[s]); mbar_arrive(&sm.raw_free[r]); }
    }
  } else if (warp == kMmaWarp) {
    // =============================== MMA issue ==================================================
    // The whole warp runs this code (operands are computed once for the warp); one elected lane, always
    // the same, issues the MMAs and the commits.
    {
      constexpr uint32_t kIdescS = idesc_f16(64, 16, 0, 0), kIdescO = idesc_f16(128, 16, 1, 1);
      const uint32_t qb = smem_u32(sm.qtile), pb = smem_u32(sm.ptile);
      auto issue_pv = [&](int i) -> bool {               // O^T += K^(first 512 dims, read along the keys) x P^T
        if (!__all_sync(0xffffffffu, mbar_wait(&sm.p_full, (uint32_t)i, abort_flag))) return false;
        fence_after_sync();
        const uint32_t kb = smem_u32(sm.khat[i % kStages]);
#pragma unroll
        for (int T = 0; T < 4; ++T)
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t ad = smem_desc(kb + T * 16 * 128 + ks * 2 * kGroupStride, kGroupStride, 128);
            const uint64_t bd = smem_desc(pb + ks * 256, 128, 1024);
            if (elect_one()) mma_f16_ss(tb + kColO + 16 * T, ad, bd, kIdescO, (i > 0 || ks > 0) ? 1u : 0u);
          }
        if (elect_one()) { commit(&sm.o_done); commit(&sm.kv_free[i % kStages]); }
        return true;
      };
      bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_ready, 0, abort_flag));
      for (int j = 0; ok && j < n_iter; ++j) {
        const int s = j % kStages;
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[s], (uint32_t)(j / kStages), abort_flag));
        if (!ok) break;
        fence_after_sync();
        const uint32_t kb = smem_u32(sm.khat[s]);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {           // S^T = K^ Q^T
          const uint64_t ad = smem_desc(kb + ks * 256, 128, kGroupStride), bd = smem_desc(qb + ks * 256, 128, kGroupStride);
          if (elect_one()) mma_f16_ss(tb + kColS + 16 * (j & 1), ad, bd, kIdescS, ks > 0);
        }
        if (elect_one()) commit(&sm.s_full[j & 1]);
        if (j > 0) ok = issue_pv(j - 1);
      }
      if (ok) issue_pv(n_iter - 1);
    }
  } else {
    // =============================== softmax warps ==============================================
    const int tq = threadIdx.x;                          // 0..127
    const uint32_t lane_addr = tb + ((uint32_t)(warp * 32) << 16);
    {
      // ---- stage the queries: bf16 -> binary16 times a power of two per head, element order (0,4,1,5,2,6,3,7) ----
      const int h = tq >> 3, sub = tq & 7;               // eight consecutive lanes share a head; words sub, sub + 8, ...
      const bool live = h < n_rep;
      const uint16_t* qrow = P.q + ((size_t)a * y.Hq + (live ? h : 0)) * kD;
      uint4 v[9];
      float mx = 0.f;
#pragma unroll
      for (int k = 0; k < 9; ++k) {
        v[k] = live ? *reinterpret_cast<const uint4*>(qrow + 8 * (sub + 8 * k)) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t u[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          mx = fmaxf(mx, fmaxf(fabsf(__uint_as_float(u[e] << 16)), fabsf(__uint_as_float(u[e] & 0xffff0000u))));
      }
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
      if (mx == 0.f) ex = 0;
      ex = min(max(ex, -100), 100);
      const float sf = __uint_as_float((uint32_t)(127 + 8 - ex) << 23);      // 256 <= max |q| * sf < 512
      if (sub == 0) sm.kappa[h] = P.scale_log2 * __uint_as_float((uint32_t)(127 - 8 + ex) << 23);
#pragma unroll
      for (int k = 0; k < 9; ++k) {
        const uint32_t u01 = v[k].x, u23 = v[k].y, u45 = v[k].z, u67 = v[k].w;
        const float x0 = __uint_as_float(u01 << 16) * sf, x1 = __uint_as_float(u01 & 0xffff0000u) * sf;
        const float x2 = __uint_as_float(u23 << 16) * sf, x3 = __uint_as_float(u23 & 0xffff0000u) * sf;
        const float x4 = __uint_as_float(u45 << 16) * sf, x5 = __uint_as_float(u45 & 0xffff0000u) * sf;
        const float x6 = __uint_as_float(u67 << 16) * sf, x7 = __uint_as_float(u67 & 0xffff0000u) * sf;
        *reinterpret_cast<uint4*>(sm.qtile + (h & 7) * 16 + (h >> 3) * kGroupStride + (sub + 8 * k) * 128) =
            make_uint4(f32x2_to_h2(x0, x4), f32x2_to_h2(x1, x5), f32x2_to_h2(x2, x6), f32x2_to_h2(x3, x7));
      }
      fence_async_smem();
      mbar_arrive(&sm.q_ready);
    }
    softmax_barrier();                                   // kappa is complete
    float kap[kHeads], m_ref[kHeads], l_part[kHeads];
#pragma unroll
    for (int h = 0; h < kHeads; ++h) { kap[h] = sm.kappa[h]; m_ref[h] = -INFINITY; l_part[h] = 0.f; }
    const bool key_lane = lane < 16;                     // an M = 64 accumulator keeps row 16 w + l in lane 32 w + l
    const int krow = warp * 16 + lane;                   // this thread's key inside the block
    bool rescaled = false;
    for (int j = 0; j < n_iter; ++j) {
      bool ok = mbar_wait(&sm.s_full[j & 1], (uint32_t)(j >> 1), abort_flag);
      fence_after_sync();
      uint32_t sr[16];
      tmem_ld16(lane_addr + kColS + 16 * (j & 1), sr);
      wait_ld();
      const int pos = (b0 + j) * 64 + krow;
      const bool valid = key_lane && pos >= lo && pos < n;
      float sc[kHeads];
      bool grow = false;
#pragma unroll
      for (int h = 0; h < kHeads; ++h) {
        sc[h] = valid ? __uint_as_float(sr[h]) * kap[h] : -INFINITY;
        grow |= sc[h] > m_ref[h] + kLazy || (m_ref[h] == -INFINITY && sc[h] != -INFINITY);
      }
      // Every softmax thread passes this barrier once per block, whatever happened to its waits; one thread samples
      // the give-up flag before it, so that all 128 leave the loop in the same block.
      if (__any_sync(0xffffffffu, grow) && lane == 0) sm.grow[j % 3] = 1;
      if (tq == 0) sm.stop[j % 3] = *abort_flag;
      softmax_barrier();
      if (tq == 0) sm.grow[(j + 2) % 3] = 0;             // not touched again before the barrier after next
      if (sm.stop[j % 3]) break;
      if (sm.grow[j % 3]) {
        // ---- exact per-head maxima of the block, new reference, rescale of what has been accumulated ----
#pragma unroll
        for (int h = 0; h < kHeads; ++h) {
          float mh = sc[h];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mh = fmaxf(mh, __shfl_xor_sync(0xffffffffu, mh, o));
          if (lane == 0) sm.wmax[warp][h] = mh;
        }
        softmax_barrier();
        float f[kHeads];
#pragma unroll
        for (int h = 0; h < kHeads; ++h) {
          const float m_new = fmaxf(fmaxf(m_ref[h], fmaxf(sm.wmax[0][h], sm.wmax[1][h])), fmaxf(sm.wmax[2][h], sm.wmax[3][h]));
          f[h] = m_new == -INFINITY ? 1.f : fast_exp2(m_ref[h] - m_new);   // m_ref = -inf: 0
          l_part[h] *= f[h];
          m_ref[h] = m_new;
        }
        if (j > 0) {
          ok = mbar_wait(&sm.o_done, (uint32_t)(j - 1), abort_flag) && ok;   // the previous value product has landed
          fence_after_sync();
#pragma unroll 1
          for (int T = 0; T < 4; ++T) {
            uint32_t orow[16];
            tmem_ld16(lane_addr + kColO + 16 * T, orow);
            wait_ld();
#pragma unroll
            for (int h = 0; h < kHeads; ++h) orow[h] = __float_as_uint(__uint_as_float(orow[h]) * f[h]);
            tmem_st16(lane_addr + kColO + 16 * T, orow);
          }
          rescaled = true;
        }
      }
      uint32_t pr[8];
#pragma unroll
      for (int h = 0; h < kHeads; h += 2) {
        const float p0 = valid ? fast_exp2(sc[h] - m_ref[h]) : 0.f;
        const float p1 = valid ? fast_exp2(sc[h + 1] - m_ref[h + 1]) : 0.f;
        l_part[h] += p0; l_part[h + 1] += p1;
        pr[h >> 1] = f32x2_to_h2(p0, p1);
      }
      // P^T is single-buffered: the previous block's value product must have read it
      if (j > 0 && !rescaled) ok = mbar_wait(&sm.o_done, (uint32_t)(j - 1), abort_flag) && ok;
      if (key_lane) {
        uint8_t* prow = sm.ptile + (krow & 7) * 16 + (krow >> 3) * 128;
        *reinterpret_cast<uint4*>(prow) = make_uint4(pr[0], pr[1], pr[2], pr[3]);
        *reinterpret_cast<uint4*>(prow + 1024) = make_uint4(pr[4], pr[5], pr[6], pr[7]);
      }
      fence_async_smem();
      if (rescaled) { wait_st(); rescaled = false; }
      fence_before_sync();
      mbar_arrive(&sm.p_full);
      (void)ok;
    }
    // ---- this share's record: acc[16][512] (unnormalised, relative to m), m, l ----
    bool fin = !*abort_flag;
    if (fin) fin = mbar_wait(&sm.o_done, (uint32_t)(n_iter - 1), abort_flag);
#pragma unroll
    for (int h = 0; h < kHeads; ++h) {
      float lh = l_part[h];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lh += __shfl_xor_sync(0xffffffffu, lh, o);
      if (lane == 0) sm.wsum[warp][h] = lh;
    }
    softmax_barrier();
    fin = __all_sync(0xffffffffu, fin && !*abort_flag);  // the loads below are warp-wide
    const bool spoiled = !fin || sm.poisoned != 0;
    if (fin) {
      fence_after_sync();
#pragma unroll 1
      for (int T = 0; T < 4; ++T) {
        uint32_t orow[16];
        tmem_ld16(lane_addr + kColO + 16 * T, orow);
        wait_ld();
        const int m = 128 * T + tq;                      // row of O^T: dim core m / 8, slot m % 8
        const int d = (m & ~7) + elem_of(m & 7);
#pragma unroll
        for (int h = 0; h < kHeads; ++h) rec[h * kRecStride + d] = spoiled ? 0.f : __uint_as_float(orow[h]);
      }
    }
    if (tq < kHeads) {
      rec[tq * kRecStride + kDv] = spoiled ? -INFINITY : m_ref[tq];
      rec[tq * kRecStride + kDv + 1] =
          spoiled ? -1.f : (sm.wsum[0][tq] + sm.wsum[1][tq]) + (sm.wsum[2][tq] + sm.wsum[3][tq]);   // negative: poisoned
    }
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
    tmem_dealloc(tb, kTmemCols);
  }
}

// grid: (16 heads, n_agents), 512 threads; combines the records of one (agent, head).  The records sit in L2 a
// microsecond away, so nothing here is a chain of dependent loads: thread s fetches (m, l) of split s, the block
// agrees on the weights, then four groups of 128 threads each take every fourth split with their loads issued
// together, and the groups' sums meet in shared memory.
constexpr int kMergeThreads = 512, kMaxSplits = 512;
__global__ void __launch_bounds__(kMergeThreads) merge_mla_kernel(int Hq, int n_splits, const float* __restrict__ records,
                                                                  void* __restrict__ out, int out_dtype,
                                                                  float* __restrict__ lse) {
  __shared__ float s_w[kMaxSplits];                      // weight of each split (0: empty)
  __shared__ float s_red[kMergeThreads / 32][2];
  __shared__ float4 s_acc[3][128];
  __shared__ float s_ml[2];
  const int h = blockIdx.x, a = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the records come from the preceding kernel
  if (h >= Hq) return;
  const float* rec = records + ((size_t)a * n_splits * kHeads + h) * kRecStride;
  const size_t step = (size_t)kHeads * kRecStride;       // between the splits of one head
  float ms = -INFINITY, ls = 0.f;
  if (tid < n_splits) { ms = rec[tid * step + kDv]; ls = rec[tid * step + kDv + 1]; }
  float M = ms, bad = ls < 0.f ? 1.f : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o)); bad = fmaxf(bad, __shfl_xor_sync(0xffffffffu, bad, o)); }
  if (lane == 0) { s_red[warp][0] = M; s_red[warp][1] = bad; }
  __syncthreads();
  M = s_red[0][0]; bad = s_red[0][1];
#pragma unroll
  for (int w = 1; w < kMergeThreads / 32; ++w) { M = fmaxf(M, s_red[w][0]); bad = fmaxf(bad, s_red[w][1]); }
  const float wgt = ms == -INFINITY ? 0.f : exp2f(ms - M);
  if (tid < n_splits) s_w[tid] = wgt;
  float L = wgt * ls;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  __syncthreads();                                       // s_red is read by everyone before it is reused
  if (lane == 0) s_red[warp][0] = L;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < kMergeThreads / 32; ++w) t += s_red[w][0];
    s_ml[0] = M; s_ml[1] = bad > 0.f ? 0.f : t;          // a poisoned split zeroes the row
  }
  const int grp = tid >> 7, d = 4 * (tid & 127);         // 128 threads x 4 consecutive dims per group
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = grp; s0 < n_splits; s0 += 16) {
    float2 lo2[4], hi2[4];
    float w4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int sp = s0 + 4 * u;
      w4[u] = sp < n_splits ? s_w[sp] : 0.f;
      lo2[u] = make_float2(0.f, 0.f); hi2[u] = make_float2(0.f, 0.f);
      if (w4[u] > 0.f) {                                 // an empty split's record holds no data
        lo2[u] = *reinterpret_cast<const float2*>(rec + sp * step + d);       // records are 8-byte aligned
        hi2[u] = *reinterpret_cast<const float2*>(rec + sp * step + d + 2);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      acc.x = fmaf(w4[u], lo2[u].x, acc.x); acc.y = fmaf(w4[u], lo2[u].y, acc.y);
      acc.z = fmaf(w4[u], hi2[u].x, acc.z); acc.w = fmaf(w4[u], hi2[u].y, acc.w);
    }
  }
  if (grp > 0) s_acc[grp - 1][tid & 127] = acc;
  __syncthreads();
  if (grp > 0) return;
  const float Lsum = s_ml[1];
  const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
#pragma unroll
  for (int g = 0; g < 3; ++g) { const float4 o = s_acc[g][tid]; acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
  acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
  const size_t out_index = ((size_t)a * Hq + h) * kDv;
  if (out_dtype == Q4KV_OUT_BF16) {
    const __nv_bfloat162 b0 = __floats2bfloat162_rn(acc.x, acc.y), b1 = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 v;
    v.x = *reinterpret_cast<const uint32_t*>(&b0);
    v.y = *reinterpret_cast<const uint32_t*>(&b1);
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + out_index + d) = v;
  } else {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + out_index + d) = acc;
  }
  if (tid == 0 && lse) lse[(size_t)a * Hq + h] = Lsum > 0.f ? (s_ml[0] + log2f(Lsum)) / kLog2e : -INFINITY;
}

struct MlaPlan { int n_splits, blocks_per_split; };
MlaPlan plan_mla(int n_agents, int max_kv_len, int window) {
  const int span = (window > 0 && window + 64 < max_kv_len) ? window + 64 : max_kv_len;
  const int blocks = (span + 63) / 64 + 1;               // a window may straddle one more 64-key block
  int n_splits = (148 + n_agents - 1) / n_agents;        // about one CTA per SM
  if (n_splits > blocks) n_splits = blocks;
  if (n_splits > kMaxSplits) n_splits = kMaxSplits;
  if (n_splits < 1) n_splits = 1;
  MlaPlan p;
  p.blocks_per_split = (blocks + n_splits - 1) / n_splits;
  p.n_splits = (blocks + p.blocks_per_split - 1) / p.blocks_per_split;
  return p;
}

}  // namespace

bool decode_mla_supported(const Layout& y) {
  return y.alias && y.D == kD && y.Dv == kDv && y.Hkv == 1 && y.Hq <= kHeads;
}

size_t decode_mla_workspace_bytes(const Layout& y, int n_agents, int max_kv_len) {
  (void)y;
  // the split count depends on the window only through a smaller span: size for the whole cache
  const MlaPlan p = plan_mla(n_agents, max_kv_len, 0);
  return (size_t)n_agents * p.n_splits * kHeads * kRecStride * sizeof(float);
}

cudaError_t launch_decode_mla(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                              const int32_t* kv_lens, int max_kv_len, int window, const void* q, float scale, void* out,
                              int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st) {
  if (b.n_agents <= 0) return cudaSuccess;
  MlaPlan plan = plan_mla(b.n_agents, max_kv_len, window);
  const MlaPlan full = plan_mla(b.n_agents, max_kv_len, 0);
  if (plan.n_splits > full.n_splits) plan = full;        // never more records than the workspace was sized for
  MlaParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.window = window;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e; P.n_splits = plan.n_splits;
  P.blocks_per_split = plan.blocks_per_split; P.records = (float*)ws; P.flags = flags;
  static bool configured[64] = {};
  const size_t smem = sizeof(MlaSmem);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(decode_mla_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(plan.n_splits, b.n_agents);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  e = cudaLaunchKernelEx(&cfg, decode_mla_kernel, P);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t mcfg = {};
  mcfg.gridDim = dim3(kHeads, b.n_agents);
  mcfg.blockDim = dim3(kMergeThreads);
  mcfg.stream = st;
  mcfg.attrs = attr;
  mcfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&mcfg, merge_mla_kernel, (int)y.Hq, plan.n_splits, (const float*)ws, out, out_dtype, lse);
}

}  // namespace q4kv
