// q4kv_decode_attention for the MLA-latent cache (d_qk = 576 = 512 latent + 64 rope, d_v = 512, V
// aliases the first 512 dims of K, one shared KV head, up to 16 query heads): one query token per
// agent in absorbed form over the Q4 latent cache, read in place (Section 3.4 "Batched Quantized
// Inference"; the MLA cache of Section 3.6).
//
// Every key serves all 16 heads and is both key and value, so the cache bytes are expanded once
// per 64-key block into a binary16 tile that the tensor cores read twice:
//   * Work is split along the keys: CTA (split, agent) walks its share of the agent's keys 64 at a
//     time (two 32-token chunks = one bulk copy of 20736 bytes into a two-slot ring, issued two
//     blocks ahead by one thread), leaves an (acc, m, l) record per head, and a second kernel combines the
//     records of an agent.
//   * The eight compute warps first turn the raw block into the tile K^ [64 keys][576 dims] in
//     shared memory (x^ = c * s + b, one binary16 fma per pair of codes, rounded once), stored as
//     8 x 16-byte core matrices: 8 keys x 8 dims each, 128 contiguous bytes -- exactly one ldmatrix
//     8x8 tile, read without bank conflicts either way.
//   * Scores: warp w owns keys 8w..8w+7 of the block: S[16 heads][8 keys] by 36 mma.sync m16n8k16
//     (A = the queries, staged once as binary16 scaled by a power of two per head; B = K^ through
//     plain ldmatrix).  Values: warp w owns dims 64w..64w+63: O[16 heads][64 dims] += P V^ by 32
//     mma.sync, with V^ = the same tile read through ldmatrix.trans and P exchanged through a 2 KB
//     shared tile.  544 tensor instructions per block over eight warps; the accumulators of the
//     whole share stay in registers.  (A tcgen05 version of this kernel was measured at 40 us per
//     call: with only 16 heads every tensor-memory MMA is tiny, and an MMA whose A operand comes
//     from shared memory costs ~110 clocks whatever its size.)
//   * Softmax with a lazily moved reference maximum per head, shared by the CTA: a block whose
//     scores exceed it by more than 2^8 triggers an exact per-head maximum (shuffles + shared
//     memory) and a rescale of the register accumulators; otherwise a block costs four
//     exponentials per thread.  Row sums stay per-thread until the end.
// Three CTA-wide named barriers per block (tile ready, growth agreed, probabilities ready); the raw
// blocks arrive on mbarriers with bounded waits (Q4KV_FLAG_INTERNAL when one runs out; the 256
// threads then leave together).  Eight warps, not nine: with a ninth the register allocation drops
// to 168 per thread, and the queries' fragments alone take 144.
#include "q4kv_layout.cuh"
#include "quantize_core.cuh"
#include "tcgen05.cuh"

namespace q4kv {

namespace {

using namespace tc;   // mbarrier and bulk-copy wrappers

constexpr int kD = 576, kDv = 512, kHeads = 16;
constexpr int kComputeWarps = 8;
constexpr int kThreads = kComputeWarps * 32;            // 256
constexpr int kChunkBytes = 32 * (kD / 2 + 4 * (kD / 64));   // 10368: [Kc 9216 | Ksb 1152]
constexpr int kRawBytes = 2 * kChunkBytes;               // one 64-key block
constexpr int kTileBytes = 64 * kD * 2;                  // 73728
constexpr int kGroupStride = (kD / 8) * 128;             // 9216: bytes between 8-row groups of a [rows][576] tile
constexpr int kStages = 2, kRawSlots = 2;
constexpr int kRecStride = kDv + 2;                      // acc[512], m, l
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLazy = 8.f;

using MlaParams = MlaDecodeParams;

struct MlaSmem {
  alignas(128) uint8_t khat[kStages][kTileBytes];        // [key 64][dim 576]: (key%8)*16 + (key/8)*9216 + (dim/8)*128
  alignas(128) uint8_t raw[kRawSlots][kRawBytes];
  alignas(128) uint8_t qtile[kHeads * kD * 2];           // [head 16][dim 576], same form
  alignas(128) uint8_t ptile[kHeads * 64 * 2];           // [head 16][key 64]: (h%8)*16 + (h/8)*1024 + (key/8)*128
  float kappa[kHeads];                                   // score in log2 units = S * kappa[head]
  float wmax[kComputeWarps][kHeads];
  float wsum[kComputeWarps][kHeads];
  alignas(8) uint64_t raw_full[kRawSlots];
  int grow[3], stop[3];
  int bad[kRawSlots];
  int abort_flag, poisoned;
  uint32_t new_words[kD / 8], new_sb[kD / 64];           // the new token's codes and (scale, bias) pairs (update-and-fetch)
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
// A bfloat16 (scale, bias) pair as a binary16 pair: exact while the magnitude is a binary16 normal number (bfloat16
// has 8 significant bits), within 2^-25 below that; a magnitude beyond binary16's largest number is reported.
__device__ inline uint32_t bf16_pair_to_h2(uint32_t u, bool& overflow) {
  const uint32_t h = f32x2_to_h2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
  overflow |= (((h & 0x7C007C00u) + 0x04000400u) & 0x80008000u) != 0u;     // an exponent field of all ones
  return h;
}
__device__ inline void compute_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }   // the eight compute warps
// four 8x8 b16 matrices; lane l supplies the address of row l % 8 of matrix l / 8; register i <- matrix i,
// thread (g, t) of the warp receiving the elements (row g, columns 2t, 2t+1)
__device__ inline void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}
// the same with every matrix transposed: thread (g, t) receives the elements (rows 2t, 2t+1, column g)
__device__ inline void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr) : "memory");
}
__device__ inline void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <bool kBf>
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
  const bool bad_len = n < 0 || n > P.len_cap;       // the host's bound on every length: the key shares cover that many keys
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
  if (threadIdx.x < 2 && threadIdx.x < n_iter)           // the first two block-table entries, fetched towards the SM meanwhile
    asm volatile("prefetch.global.L1 [%0];" ::"l"(P.tables + (size_t)a * P.max_blocks + ((2 * (b0 + (int)threadIdx.x)) >> 3)) : "memory");
  // While the preceding kernel drains, L2 is asked for the agent's query rows (a prefetch returns nothing to the kernel,
  // so it may precede the wait; in a decode step they are what the preceding kernels have just written).
  {
    const int lines = n_rep * kD * 2 / 128;                // 128-byte lines of the agent's n_rep query rows
    const uint16_t* qrows = P.q + (size_t)a * y.Hq * kD;
    for (int i = threadIdx.x; i < lines; i += kThreads) asm volatile("prefetch.global.L2 [%0];" ::"l"(qrows + i * 64));
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the new token was appended by the preceding kernel
  volatile int* abort_flag = &sm.abort_flag;

  // Raw 64-key blocks: one bulk copy each into a two-slot ring, issued by thread 0 -- blocks 0 and 1 here, block
  // j + 2 once every warp has left block j's raw bytes (the barrier after the dequantize step).
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
    issue_block(0);
    if (n_iter > 1) issue_block(1);
    issued = min(n_iter, kRawSlots);
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
      const QuantOut qo = quantize_eight(x, kBf);             // eight lanes per group of 64; 72 words = 9 whole groups
      if (w < kD / 8) {
        sm.new_words[w] = qo.word;
        if ((w & 7) == 0) sm.new_sb[w >> 3] = *reinterpret_cast<const uint32_t*>(&qo.sb);
      }
    }
  }

  // =============================== compute warps ================================================
  const int tq = threadIdx.x;                            // 0..255
  const int g = lane >> 2, tid = lane & 3;               // fragment coordinates
  {
    // ---- stage the queries: bf16 -> binary16 times a power of two per head, element order (0,4,1,5,2,6,3,7) ----
    const int h = tq >> 4, sub = tq & 15;                // sixteen consecutive lanes share a head; words sub, sub + 16, ...
    const bool live = h < n_rep;
    const uint16_t* qrow = P.q + ((size_t)a * y.Hq + (live ? h : 0)) * kD;
    uint4 v[5];
    float mx = 0.f;
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const int w = sub + 16 * k;
      v[k] = (live && w < kD / 8) ? *reinterpret_cast<const uint4*>(qrow + 8 * w) : make_uint4(0u, 0u, 0u, 0u);
      const uint32_t u[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
        mx = fmaxf(mx, fmaxf(fabsf(__uint_as_float(u[e] << 16)), fabsf(__uint_as_float(u[e] & 0xffff0000u))));
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
    if (mx == 0.f) ex = 0;
    ex = min(max(ex, -100), 100);
    const float sf = __uint_as_float((uint32_t)(127 + 8 - ex) << 23);        // 256 <= max |q| * sf < 512
    if (sub == 0) sm.kappa[h] = P.scale_log2 * __uint_as_float((uint32_t)(127 - 8 + ex) << 23);
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const int w = sub + 16 * k;
      if (w >= kD / 8) continue;
      const uint32_t u01 = v[k].x, u23 = v[k].y, u45 = v[k].z, u67 = v[k].w;
      const float x0 = __uint_as_float(u01 << 16) * sf, x1 = __uint_as_float(u01 & 0xffff0000u) * sf;
      const float x2 = __uint_as_float(u23 << 16) * sf, x3 = __uint_as_float(u23 & 0xffff0000u) * sf;
      const float x4 = __uint_as_float(u45 << 16) * sf, x5 = __uint_as_float(u45 & 0xffff0000u) * sf;
      const float x6 = __uint_as_float(u67 << 16) * sf, x7 = __uint_as_float(u67 & 0xffff0000u) * sf;
      *reinterpret_cast<uint4*>(sm.qtile + (h & 7) * 16 + (h >> 3) * kGroupStride + w * 128) =
          make_uint4(f32x2_to_h2(x0, x4), f32x2_to_h2(x1, x5), f32x2_to_h2(x2, x6), f32x2_to_h2(x3, x7));
    }
  }
  compute_barrier();                                     // queries and kappa are complete

  // per-chunk dequantize coordinates: thread xx of 128 owns token tau = 4 kg + ki of chunk ci and, of its 72 words,
  // those with w % 4 == kt (four 16-byte pieces and one 8-byte piece).  The eight lanes of a shared-memory phase
  // read eight different 16-byte columns and write eight different rows.
  const int ci = tq >> 7, xx = tq & 127;
  const int ki = xx & 3, kg = 2 * ((xx >> 3) & 3) + ((xx >> 2) & 1), kt = (ki + (xx >> 5)) & 3;
  const int tau = 4 * kg + ki;
  const int rd16 = ci * kChunkBytes + (ki * 144 + kg * 4 + kt) * 16;        // + j * 512
  const int rd8 = ci * kChunkBytes + (ki * 576 + 512) * 4 + (kg * 4 + kt) * 8;
  const int sb_at = ci * kChunkBytes + 9216 + ((((tau & 3) * 4 + (tau >> 3)) * 2 + ((tau >> 2) & 1)) * 9) * 4;   // + 4 * group
  const int krow = ci * 32 + tau;
  const int wr_at = (krow & 7) * 16 + (krow >> 3) * kGroupStride + kt * 128;

  // ldmatrix lane addresses (lane l: matrix l / 8, row l % 8)
  const int lm = lane >> 3, lr = lane & 7;
  const uint32_t q_lane = smem_u32(sm.qtile) + lr * 16 + (lm & 1) * kGroupStride + (lm >> 1) * 128;   // + 256 per k-step
  const uint32_t p_lane = smem_u32(sm.ptile) + lr * 16 + (lm & 1) * 1024 + (lm >> 1) * 128;           // + 256 per k-step
  const uint32_t kq_lane = lr * 16 + warp * kGroupStride + lm * 128;        // scores: key octet = warp; + 512 per two k-steps
  const uint32_t kv_lane = lr * 16 + (lm & 1) * kGroupStride + (8 * warp + (lm >> 1)) * 128;   // values: + 2 ks octets, + 256 per dim-core pair

  // The queries never change: their A fragments (36 k-steps x 4 registers) live in registers for the whole launch.
  uint32_t qa[kD / 16][4];
#pragma unroll
  for (int ks = 0; ks < kD / 16; ++ks) ldmatrix_x4(qa[ks], q_lane + ks * 256);
  float kap[2], m_ref[2], l_part[2];                     // heads g and g + 8
  kap[0] = sm.kappa[g]; kap[1] = sm.kappa[g + 8];
  m_ref[0] = -INFINITY; m_ref[1] = -INFINITY; l_part[0] = 0.f; l_part[1] = 0.f;
  float o[8][4];                                         // [dim core 8 warp + c][head g: slots 2 tid, 2 tid + 1 | head g + 8: same]
#pragma unroll
  for (int c = 0; c < 8; ++c) { o[c][0] = 0.f; o[c][1] = 0.f; o[c][2] = 0.f; o[c][3] = 0.f; }

  bool stopped = false;
  for (int j = 0; j < n_iter; ++j) {
    const int s = j % kStages, r = j % kRawSlots;
    // ---- raw block -> binary16 tile (every thread: one token of one chunk, 18 words) ----
    mbar_wait(&sm.raw_full[r], (uint32_t)(j / kRawSlots), abort_flag);     // a wait that runs out raises the give-up flag
    if (has_new && j == n_iter - 1) {
      // words 0..71 and the nine (scale, bias) pairs of position n - 1, one per thread
      if (sm.bad[r] == 0 && tq < kD / 8 + kD / 64) {
        const int tau_n = (n - 1) & 31, c = 2 * (b0 + j);
        const uint32_t at = (uint32_t)(((n - 1) >> 5) & 1) * kChunkBytes +
                            (tq < kD / 8 ? y.off_kc + 4u * k_word_offset(tau_n, tq, kD / 64)
                                         : y.off_ksb + 4u * sb_offset(tau_n, tq - kD / 8, kD / 64));
        const uint32_t val = tq < kD / 8 ? sm.new_words[tq] : sm.new_sb[tq - kD / 8];
        *reinterpret_cast<uint32_t*>(sm.raw[r] + at) = val;
        const int blk = P.tables[(size_t)a * P.max_blocks + (c >> 3)];      // checked when the copy was issued
        // the caller of the update-and-fetch entry owns the pool for writing
        uint8_t* dst = const_cast<uint8_t*>(head_block(P.pool, y, P.layer, blk, 0)) + (size_t)(c & 7) * kChunkBytes + at;
        *reinterpret_cast<uint32_t*>(dst) = val;
      }
      compute_barrier();
    }
    if (kBf) {
      // bfloat16 scales and biases become binary16 in place, once per block (the tile is binary16); only the tokens
      // below the agent's length count for the range report (bytes past the end are whatever was there)
      bool overflow = false;
      for (int w = tq; w < 2 * 288; w += kThreads) {     // per chunk: 32 tokens x 9 groups
        const int cw = w >= 288 ? 1 : 0, o = w - 288 * cw;
        const int row = o / 9;                           // (i * 4 + tid) * 2 + e: token 8 tid + 4 e + i
        const int tok = 8 * ((row >> 1) & 3) + 4 * (row & 1) + (row >> 3);
        uint32_t* at = reinterpret_cast<uint32_t*>(sm.raw[r] + cw * kChunkBytes + 9216 + 4 * o);
        bool over = false;
        *at = bf16_pair_to_h2(*at, over);
        overflow |= over && (b0 + j) * 64 + cw * 32 + tok < n;
      }
      if (overflow && sm.bad[r] == 0) raise_flag(P.flags, Q4KV_FLAG_SB_RANGE);
      compute_barrier();
    }
    {
      const uint8_t* raw = sm.raw[r];
      const bool dead = sm.bad[r] != 0 || (b0 + j) * 64 + krow >= n;       // stale bytes past the end
      uint8_t* dst = sm.khat[s] + wr_at;
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const uint4 kw = *reinterpret_cast<const uint4*>(raw + rd16 + jj * 512);
        uint32_t sb0 = *reinterpret_cast<const uint32_t*>(raw + sb_at + 8 * jj);            // group 2 jj
        uint32_t sb1 = *reinterpret_cast<const uint32_t*>(raw + sb_at + 8 * jj + 4);        // group 2 jj + 1
        if (dead) { sb0 = 0u; sb1 = 0u; }
        const uint32_t s0 = __byte_perm(sb0, sb0, 0x1010), c0 = __byte_perm(sb0, sb0, 0x3232);
        const uint32_t s1 = __byte_perm(sb1, sb1, 0x1010), c1 = __byte_perm(sb1, sb1, 0x3232);
        *reinterpret_cast<uint4*>(dst + (16 * jj + 0) * 128) = dequant8(kw.x, s0, c0);
        *reinterpret_cast<uint4*>(dst + (16 * jj + 4) * 128) = dequant8(kw.y, s0, c0);
        *reinterpret_cast<uint4*>(dst + (16 * jj + 8) * 128) = dequant8(kw.z, s1, c1);
        *reinterpret_cast<uint4*>(dst + (16 * jj + 12) * 128) = dequant8(kw.w, s1, c1);
      }
      {
        const uint2 kw = *reinterpret_cast<const uint2*>(raw + rd8);
        uint32_t sb8 = *reinterpret_cast<const uint32_t*>(raw + sb_at + 32);                // group 8
        if (dead) sb8 = 0u;
        const uint32_t s8 = __byte_perm(sb8, sb8, 0x1010), c8 = __byte_perm(sb8, sb8, 0x3232);
        *reinterpret_cast<uint4*>(dst + 64 * 128) = dequant8(kw.x, s8, c8);
        *reinterpret_cast<uint4*>(dst + 68 * 128) = dequant8(kw.y, s8, c8);
      }
    }
    if (tq == 0) sm.stop[j % 3] = *abort_flag;           // sampled by one thread: all 256 leave in the same block
    compute_barrier();                                   // the tile is complete, and nobody reads the raw slot any more
    if (sm.stop[j % 3]) { stopped = true; break; }
    if (tq == 0 && j + kRawSlots < n_iter) { issue_block(j + kRawSlots); issued = j + kRawSlots + 1; }

    // ---- scores of this warp's eight keys: S[16 heads][8 keys], 36 k-steps ----
    float sc[4];
    {
      // four independent accumulation chains (the tensor instruction's latency, not its rate, would bound one chain)
      float acc[4][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { acc[i][0] = 0.f; acc[i][1] = 0.f; acc[i][2] = 0.f; acc[i][3] = 0.f; }
      const uint32_t kb = smem_u32(sm.khat[s]) + kq_lane;
#pragma unroll
      for (int kk = 0; kk < kD / 32; ++kk) {
        uint32_t bq[4];
        ldmatrix_x4(bq, kb + kk * 512);
        mma_f16(acc[(2 * kk) & 3], qa[2 * kk], bq[0], bq[1]);
        mma_f16(acc[(2 * kk + 1) & 3], qa[2 * kk + 1], bq[2], bq[3]);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[e] = (acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e]);
    }
    // this thread: heads g (sc[0], sc[1]) and g + 8 (sc[2], sc[3]), keys 8 warp + 2 tid, + 1
    const int pos = (b0 + j) * 64 + 8 * warp + 2 * tid;
    const bool v0 = pos >= lo && pos < n, v1 = pos + 1 >= lo && pos + 1 < n;
    sc[0] = v0 ? sc[0] * kap[0] : -INFINITY; sc[1] = v1 ? sc[1] * kap[0] : -INFINITY;
    sc[2] = v0 ? sc[2] * kap[1] : -INFINITY; sc[3] = v1 ? sc[3] * kap[1] : -INFINITY;
    const float mx0 = fmaxf(sc[0], sc[1]), mx1 = fmaxf(sc[2], sc[3]);
    const bool grow = mx0 > m_ref[0] + kLazy || (m_ref[0] == -INFINITY && mx0 != -INFINITY) ||
                      mx1 > m_ref[1] + kLazy || (m_ref[1] == -INFINITY && mx1 != -INFINITY);
    if (__any_sync(0xffffffffu, grow) && lane == 0) sm.grow[j % 3] = 1;
    compute_barrier();                                   // growth agreed (and every warp has left the previous block's P)
    if (tq == 0) sm.grow[(j + 2) % 3] = 0;               // not touched again before the barrier after next
    if (sm.grow[j % 3]) {
      // ---- exact per-head maxima of the block, new reference, rescale of what has been accumulated ----
      float w0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)), w1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      w0 = fmaxf(w0, __shfl_xor_sync(0xffffffffu, w0, 2)); w1 = fmaxf(w1, __shfl_xor_sync(0xffffffffu, w1, 2));
      if (tid == 0) { sm.wmax[warp][g] = w0; sm.wmax[warp][g + 8] = w1; }
      compute_barrier();
      float f[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float m_new = m_ref[e];
#pragma unroll
        for (int w = 0; w < kComputeWarps; ++w) m_new = fmaxf(m_new, sm.wmax[w][g + 8 * e]);
        f[e] = m_new == -INFINITY ? 1.f : fast_exp2(m_ref[e] - m_new);     // m_ref = -inf: 0
        l_part[e] *= f[e];
        m_ref[e] = m_new;
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) { o[c][0] *= f[0]; o[c][1] *= f[0]; o[c][2] *= f[1]; o[c][3] *= f[1]; }
    }
    // ---- probabilities (a head without any key yet keeps the reference at -inf and p = 0) ----
    const float p0 = v0 ? fast_exp2(sc[0] - m_ref[0]) : 0.f, p1 = v1 ? fast_exp2(sc[1] - m_ref[0]) : 0.f;
    const float p2 = v0 ? fast_exp2(sc[2] - m_ref[1]) : 0.f, p3 = v1 ? fast_exp2(sc[3] - m_ref[1]) : 0.f;
    l_part[0] += p0 + p1; l_part[1] += p2 + p3;
    *reinterpret_cast<uint32_t*>(sm.ptile + (g & 7) * 16 + 0 * 1024 + warp * 128 + 4 * tid) = f32x2_to_h2(p0, p1);
    *reinterpret_cast<uint32_t*>(sm.ptile + (g & 7) * 16 + 1 * 1024 + warp * 128 + 4 * tid) = f32x2_to_h2(p2, p3);
    compute_barrier();                                   // the probabilities of all 64 keys are in place

    // ---- values: O[16 heads][dims 64 warp ..] += P V^, four k-steps of 16 keys ----
    {
      const uint32_t vb = smem_u32(sm.khat[s]) + kv_lane;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        uint32_t pa[4];
        ldmatrix_x4(pa, p_lane + ks * 256);
#pragma unroll
        for (int c = 0; c < 8; c += 2) {
          uint32_t bv[4];
          ldmatrix_x4_trans(bv, vb + ks * 2 * kGroupStride + c * 128);
          mma_f16(o[c], pa, bv[0], bv[1]);
          mma_f16(o[c + 1], pa, bv[2], bv[3]);
        }
      }
    }
  }

  // ---- this share's record: acc[16][512] (unnormalised, relative to m), m, l ----
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float lh = l_part[e];
    lh += __shfl_xor_sync(0xffffffffu, lh, 1);
    lh += __shfl_xor_sync(0xffffffffu, lh, 2);
    if (tid == 0) sm.wsum[warp][g + 8 * e] = lh;
  }
  compute_barrier();
  const bool spoiled = stopped || sm.poisoned != 0;
  if (stopped && tq == 0) {
    // giving up: let the copies that may still be in flight land before shared memory is released
    for (int jj = max(0, issued - kRawSlots); jj < issued; ++jj)
      for (uint32_t i = 0; i < 64 && !mbar_try_wait(&sm.raw_full[jj % kRawSlots], (uint32_t)(jj / kRawSlots) & 1u); ++i) {}
    raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    // dim core 8 warp + c, slots 2 tid and 2 tid + 1 of its 16-byte row
    const int d0 = 8 * (8 * warp + c) + elem_of(2 * tid), d1 = 8 * (8 * warp + c) + elem_of(2 * tid + 1);
    rec[g * kRecStride + d0] = spoiled ? 0.f : o[c][0];
    rec[g * kRecStride + d1] = spoiled ? 0.f : o[c][1];
    rec[(g + 8) * kRecStride + d0] = spoiled ? 0.f : o[c][2];
    rec[(g + 8) * kRecStride + d1] = spoiled ? 0.f : o[c][3];
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

// grid: (16 heads, n_agents, 4 quarters of the value dims), 512 threads; combines the records of one (agent, head)
// for 128 output dims.  The records sit in L2 a microsecond away, so nothing here is a chain of dependent loads: thread
// s fetches (m, l) of split s, the block agrees on the weights, while sixteen groups of 32 threads each take every
// sixteenth split with their loads issued together (up to 64 splits are in flight before the weights are known),
// and the groups' sums meet in shared memory.  Four CTAs per (agent, head) rather than one: a quarter of the record
// bytes per CTA and four times the SMs pulling them (4.1 -> see the profile).
constexpr int kMergeThreads = 512, kMaxSplits = 512, kMergeGroups = kMergeThreads / 32, kMergeQuarters = 4;
__global__ void __launch_bounds__(kMergeThreads) merge_mla_kernel(int Hq, int n_splits, const float* __restrict__ records,
                                                                  void* __restrict__ out, int out_dtype,
                                                                  float* __restrict__ lse) {
  __shared__ float s_w[kMaxSplits];                      // weight of each split (0: empty)
  __shared__ float s_red[kMergeThreads / 32][2];
  __shared__ float4 s_acc[kMergeGroups - 1][32];
  __shared__ float s_ml[2];
  const int h = blockIdx.x, a = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");     // the records come from the preceding kernel
  if (h >= Hq) return;
  const float* rec = records + ((size_t)a * n_splits * kHeads + h) * kRecStride;
  const size_t step = (size_t)kHeads * kRecStride;       // between the splits of one head
  // The record loads of the first 16 * kPre splits do not wait for the weights: they are issued first and overlap the
  // round trip of the (m, l) loads (an empty split's data is whatever an earlier call left there; it is dropped below).
  constexpr int kPre = 4;
  const int grp = warp, d = (kDv / kMergeQuarters) * blockIdx.z + 4 * lane;   // 32 lanes x 4 consecutive dims per group
  float4 pre[kPre];
#pragma unroll
  for (int u = 0; u < kPre; ++u) {
    const int sp = grp + kMergeGroups * u;
    pre[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (sp < n_splits) {
      const float2 lo2 = *reinterpret_cast<const float2*>(rec + sp * step + d);       // records are 8-byte aligned
      const float2 hi2 = *reinterpret_cast<const float2*>(rec + sp * step + d + 2);
      pre[u] = make_float4(lo2.x, lo2.y, hi2.x, hi2.y);
    }
  }
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
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int u = 0; u < kPre; ++u) {
    const int sp = grp + kMergeGroups * u;
    const float wu = sp < n_splits ? s_w[sp] : 0.f;
    if (wu > 0.f) {                                      // an empty split's record holds no data
      acc.x = fmaf(wu, pre[u].x, acc.x); acc.y = fmaf(wu, pre[u].y, acc.y);
      acc.z = fmaf(wu, pre[u].z, acc.z); acc.w = fmaf(wu, pre[u].w, acc.w);
    }
  }
  for (int sp = grp + kMergeGroups * kPre; sp < n_splits; sp += kMergeGroups) {
    const float wu = s_w[sp];
    if (wu > 0.f) {
      const float2 lo2 = *reinterpret_cast<const float2*>(rec + sp * step + d);
      const float2 hi2 = *reinterpret_cast<const float2*>(rec + sp * step + d + 2);
      acc.x = fmaf(wu, lo2.x, acc.x); acc.y = fmaf(wu, lo2.y, acc.y);
      acc.z = fmaf(wu, hi2.x, acc.z); acc.w = fmaf(wu, hi2.y, acc.w);
    }
  }
  if (grp > 0) s_acc[grp - 1][lane] = acc;
  __syncthreads();
  if (grp > 0) return;
  const float Lsum = s_ml[1];
  const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
#pragma unroll
  for (int g = 0; g < kMergeGroups - 1; ++g) { const float4 o = s_acc[g][lane]; acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
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
  if (tid == 0 && blockIdx.z == 0 && lse) lse[(size_t)a * Hq + h] = Lsum > 0.f ? (s_ml[0] + log2f(Lsum)) / kLog2e : -INFINITY;
}

struct MlaPlan { int n_splits, blocks_per_split; };
MlaPlan plan_mla(int n_agents, int max_kv_len, int window) {
  const int span = (window > 0 && window + 64 < max_kv_len) ? window + 64 : max_kv_len;
  const int blocks = (span + 63) / 64 + 1;               // a window may straddle one more 64-key block
  int n_splits = (sm_count() + n_agents - 1) / n_agents;   // about one CTA per SM
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
                              int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st, const void* k_new,
                              bool on_codes) {
  if (b.n_agents <= 0) return cudaSuccess;
  MlaPlan plan = plan_mla(b.n_agents, max_kv_len, window);
  const MlaPlan full = plan_mla(b.n_agents, max_kv_len, 0);
  if (plan.n_splits > full.n_splits) plan = full;        // never more records than the workspace was sized for
  MlaParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.len_cap = max_kv_len; P.window = window;
  P.q = (const uint16_t*)q; P.k_new = (const uint16_t*)k_new; P.scale_log2 = scale * kLog2e; P.n_splits = plan.n_splits;
  P.blocks_per_split = plan.blocks_per_split; P.records = (float*)ws; P.flags = flags;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaError_t e;
  if (on_codes) {
    e = launch_mla_codes_kernel(P, st);
  } else {
    static bool configured[64][2] = {};
    const size_t smem = sizeof(MlaSmem);
    const int bf = y.sb_bf16 ? 1 : 0;
    void (*kernel)(const MlaParams) = bf ? decode_mla_kernel<true> : decode_mla_kernel<false>;
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev][bf]) {
      e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) configured[dev][bf] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.n_splits, b.n_agents);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, P);
  }
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t mcfg = {};
  mcfg.gridDim = dim3(kHeads, b.n_agents, kMergeQuarters);
  mcfg.blockDim = dim3(kMergeThreads);
  mcfg.stream = st;
  mcfg.attrs = attr;
  mcfg.numAttrs = 1;
  return cudaLaunchKernelEx(&mcfg, merge_mla_kernel, (int)y.Hq, plan.n_splits, (const float*)ws, out, out_dtype, lse);
}

}  // namespace q4kv
