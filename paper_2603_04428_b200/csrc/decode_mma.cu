// q4kv_decode_attention, tensor-core path for GQA shapes (d_qk = d_v in {128, 256}, at most four
// query heads per KV head): one query token per agent over its whole Q4 cache, read in place
// (Section 3.4 "Batched Quantized Inference": fused attention on the Q4 tensors; Section 3.6:
// GQA head mapping and sliding-window layers).
//
// The kernel is bound by HBM bandwidth, so it is organised around the byte stream:
//   * Work = the flattened list of 32-token chunks of all (agent, KV head) pairs inside their key
//     range [lo, kv_len).  The list is cut into equal contiguous ranges, one per persistent CTA,
//     so ragged lengths balance by construction.  A CTA's range may cover parts of several
//     pairs ("segments"); per segment it writes one partial (m, l, acc) record and a small
//     second kernel combines the records of each pair.
//   * A producer warp streams the CTA's chunks through a shared-memory ring with one bulk
//     asynchronous copy per chunk (a chunk is one contiguous byte range of the pool) completing
//     on an mbarrier; four consumer warps take chunks round-robin.
//   * Arithmetic runs on the 4-bit codes, not on dequantized values.  With x^ = c*s + b and one
//     (s, b) per token and 64-element group,
//         q.k_t   = sum_g [ s_tg * (sum_{d in g} q_d c_td) + b_tg * (sum_{d in g} q_d) ]
//         (p.V)_d = sum_t (p_t s_tg(d)) c_td + sum_t p_t b_tg(d),
//     so both contractions are mma.sync m16n8k16 (f16 in, f32 accumulate) whose code operand is
//     produced by masking the packed word: a nibble in the low bits of a 16-bit lane is the
//     binary16 subnormal c * 2^-24 (or 16c * 2^-24 one nibble higher; the 16 is folded into the
//     other operand), which the tensor cores multiply exactly.  Cost: 5 logic ops per 8 codes.
//   * Scores come out as [8 query rows x 8 tokens] fragments whose lane ownership is exactly the
//     B-operand ownership of the P.V product, so probabilities never move between lanes.  Rows
//     4..7 repeat the (at most four) query heads: they carry the low half of a two-term binary16
//     split of p*s, which makes the value product accurate to ~2^-22 at no extra MMA.
#include "q4kv_layout.cuh"

namespace q4kv {

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;       // + one producer warp
constexpr int kCtasPerSm = 2;
constexpr int kRingBytes = 73728;                      // 16 chunks at d = 128, 8 at d = 256
constexpr uint32_t kSpinLimit = 1u << 22;              // bounded mbarrier waits (each try blocks a while in hardware)
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kMaskLo = 0x000F000Fu, kMaskHi = 0x00F000F0u;

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
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
// Bounded wait: gives up after kSpinLimit tries or as soon as another warp has given up.
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
__device__ inline void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

__device__ inline void mma16816(float c[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ inline float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ inline uint32_t h2_bits(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ inline float2 h2_to_f2(uint32_t u) { return __half22float2(*reinterpret_cast<__half2*>(&u)); }

// ---------------------------------------------------------------------------------------------
// Work list: chunks of all (agent, KV head) pairs, agent-major, then head, then chunk
// ---------------------------------------------------------------------------------------------
struct AgentRange { int n, lo, cf, nc; };   // keys [lo, n); chunks cf .. cf+nc-1

__device__ inline AgentRange agent_range(const int32_t* __restrict__ kv_lens, int a, int window, int max_blocks,
                                         bool& bad) {
  AgentRange r;
  r.n = kv_lens[a];
  bad = r.n < 0 || r.n > max_blocks * kBlockTokens;
  if (bad) r.n = 0;
  r.lo = window > 0 ? max(0, r.n - window) : 0;
  r.cf = r.lo >> 5;
  r.nc = r.n > r.lo ? ((r.n + 31) >> 5) - r.cf : 0;
  return r;
}

// Warp-cooperative pass over the agents.  Returns the total number of units; when `want` >= 0
// also locates the agent containing unit `want` (agent index, first unit of that agent).
__device__ inline long long scan_units(const int32_t* __restrict__ kv_lens, int n_agents, int Hkv, int window,
                                       int max_blocks, long long want, int& agent, long long& agent_start,
                                       bool& any_bad) {
  const int lane = threadIdx.x & 31;
  long long cum = 0;
  agent = -1;
  agent_start = 0;
  any_bad = false;
  for (int base = 0; base < n_agents; base += 32) {
    const int a = base + lane;
    long long cnt = 0;
    bool bad = false;
    if (a < n_agents) cnt = (long long)agent_range(kv_lens, a, window, max_blocks, bad).nc * Hkv;
    any_bad |= __any_sync(0xffffffffu, bad);
    long long inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const long long tot = __shfl_sync(0xffffffffu, inc, 31);
    if (agent < 0 && want >= 0 && want < cum + tot) {
      const unsigned bal = __ballot_sync(0xffffffffu, cum + inc > want);
      const int l = __ffs(bal) - 1;
      agent = base + l;
      agent_start = cum + __shfl_sync(0xffffffffu, inc, l) - __shfl_sync(0xffffffffu, cnt, l);
    }
    cum += tot;
  }
  return cum;
}

__device__ inline long long range_begin(long long U, int c, int n_ctas) { return U * c / n_ctas; }
__device__ inline int cta_of_unit(long long U, long long u, int n_ctas) {
  int c = (int)(u * n_ctas / U);
  while (c + 1 < n_ctas && range_begin(U, c + 1, n_ctas) <= u) ++c;
  return c;
}

// One segment: the part of pair (agent a, KV head hk) inside this CTA's unit range.
struct Segment {
  int a, hk, c0, c1;      // logical chunk indices [c0, c1) of the agent
  int n, lo;              // key range of the agent
  long long k0;           // running chunk counter of the CTA at c0
  long long u0;           // global unit index at c0
  bool first_of_pair;     // c0 is the pair's first chunk
};

struct Walker {
  const int32_t* kv_lens;
  int n_agents, Hkv, window, max_blocks;
  long long u, u_end, k;
  int a, hk, c;
  AgentRange r;

  __device__ void init(const int32_t* kv_lens_, int n_agents_, int Hkv_, int window_, int max_blocks_, long long u_begin,
                       long long u_end_, int agent, long long agent_start) {
    kv_lens = kv_lens_; n_agents = n_agents_; Hkv = Hkv_; window = window_; max_blocks = max_blocks_;
    u = u_begin; u_end = u_end_; k = 0;
    a = agent;
    if (u < u_end && a >= 0) {
      bool bad;
      r = agent_range(kv_lens, a, window, max_blocks, bad);
      const long long rem = u - agent_start;
      hk = (int)(rem / r.nc);
      c = r.cf + (int)(rem % r.nc);
    }
  }
  __device__ bool next(Segment& s) {
    if (u >= u_end || a < 0) return false;
    const int pair_end = r.cf + r.nc;
    const long long left = u_end - u;
    const int c1 = (long long)(pair_end - c) <= left ? pair_end : c + (int)left;
    s.a = a; s.hk = hk; s.c0 = c; s.c1 = c1; s.n = r.n; s.lo = r.lo; s.k0 = k; s.u0 = u;
    s.first_of_pair = (c == r.cf);
    const int cnt = c1 - c;
    u += cnt; k += cnt;
    if (c1 == pair_end) {
      ++hk;
      if (hk == Hkv) {
        hk = 0;
        bool bad;
        do {
          ++a;
          if (a >= n_agents) { a = -1; break; }
          r = agent_range(kv_lens, a, window, max_blocks, bad);
        } while (r.nc == 0);
      }
      if (a >= 0) c = r.cf;
    } else {
      c = c1;
    }
    return true;
  }
};

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
struct DecodeParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks;
  const int32_t* tables;
  const int32_t* kv_lens;
  int window;
  const uint16_t* q;          // bf16 [A][Hq][D]
  float scale_log2;           // softmax_scale * log2(e)
  int2* desc;                 // [A*Hkv] (first CTA, last CTA) of each non-empty pair
  float* partials;            // [A*Hkv + n_ctas][n_rep][Dv + 2]
  int32_t* flags;
};

template <int G>
struct Smem {
  static constexpr int D = 64 * G;
  static constexpr int kChunkBytes = 32 * (D / 2 + 4 * G) * 2;
  static constexpr int kSlots = kRingBytes / kChunkBytes;
  static constexpr int kMergeStride = D + 8;            // acc[Dv], m, l, bias[Gv], pad
  alignas(128) uint8_t ring[kSlots * kChunkBytes];
  alignas(8) uint64_t full[kSlots];
  uint64_t empty[kSlots];
  int bad[kSlots];
  int abort_flag;
  alignas(16) __half qh[4][D];          // normalized query rows (odd dims pre-divided by 16)
  float qsum[4][G];                     // scale_log2 * sum of the true q over each group
  float kappa[4];                       // scale_log2 * 2^(24 + E - 10)
  alignas(16) float merge[kConsumerWarps][4][kMergeStride];
};

template <int G>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) decode_mma_kernel(const DecodeParams P) {
  constexpr int D = 64 * G, Dv = D, Gv = G;
  using S = Smem<G>;
  constexpr int kSlots = S::kSlots, kChunkBytes = S::kChunkBytes;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  S& sm = *reinterpret_cast<S*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const int n_rep = y.n_rep;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); sm.bad[s] = 0; }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  // ---- this CTA's unit range (every warp computes it for itself) ----
  int agent0;
  long long agent0_start;
  bool any_bad;
  const long long U = scan_units(P.kv_lens, P.n_agents, y.Hkv, P.window, P.max_blocks, -1, agent0, agent0_start, any_bad);
  if (any_bad && cta == 0 && threadIdx.x == 0) raise_flag(P.flags, Q4KV_FLAG_BAD_LENGTH);
  if (U == 0) return;
  // never more ranges than units: every CTA below n_ctas then owns a non-empty range
  const int n_ctas = (long long)gridDim.x < U ? (int)gridDim.x : (int)U;
  if (cta >= n_ctas) return;
  const long long u_begin = range_begin(U, cta, n_ctas), u_end = range_begin(U, cta + 1, n_ctas);
  if (u_begin >= u_end) return;
  scan_units(P.kv_lens, P.n_agents, y.Hkv, P.window, P.max_blocks, u_begin, agent0, agent0_start, any_bad);
  Walker wk;
  wk.init(P.kv_lens, P.n_agents, y.Hkv, P.window, P.max_blocks, u_begin, u_end, agent0, agent0_start);
  Segment seg;

  // =============================== producer warp ===============================================
  if (warp == kConsumerWarps) {
    if (lane != 0) return;
    while (wk.next(seg)) {
      int cached_lb = -1, blk = -1;
      for (int c = seg.c0; c < seg.c1; ++c) {
        const long long k = seg.k0 + (c - seg.c0);
        const int slot = (int)(k % kSlots);
        const uint32_t round = (uint32_t)(k / kSlots);
        if (round > 0 && !mbar_wait(&sm.empty[slot], (round - 1) & 1u, &sm.abort_flag)) {
          raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
          return;
        }
        if ((c >> 3) != cached_lb) {
          cached_lb = c >> 3;
          blk = P.tables[(size_t)seg.a * P.max_blocks + cached_lb];
        }
        if (blk < 0 || blk >= P.n_blocks) {
          sm.bad[slot] = 1;
          raise_flag(P.flags, Q4KV_FLAG_BAD_BLOCK);
          mbar_arrive(&sm.full[slot]);
        } else {
          sm.bad[slot] = 0;
          mbar_arrive_expect_tx(&sm.full[slot], kChunkBytes);
          bulk_load(sm.ring + (size_t)slot * kChunkBytes,
                    head_block(P.pool, y, P.layer, blk, seg.hk) + (size_t)(c & 7) * kChunkBytes, kChunkBytes,
                    &sm.full[slot]);
        }
      }
    }
    return;
  }

  // =============================== consumer warps ==============================================
  const int g = lane >> 2, tid = lane & 3;
  const int hrow = g & 3;                              // query head (within the KV head) of this lane's score row
  const float delta = g >= 4 ? 1.f : 0.f;              // rows 4..7 carry the low half of the p*s split
  bool aborted = false;

  while (wk.next(seg)) {
    // ---- stage the query rows of this pair: normalize by a power of two, sums per group ----
    if (warp < n_rep) {
      const uint16_t* qrow = P.q + ((size_t)seg.a * y.Hq + (size_t)seg.hk * n_rep + warp) * D;
      constexpr int E = D / 32;                        // elements per lane (4 or 8), all in one group
      float x[E];
      if (E == 4) {
        const uint2 v = *reinterpret_cast<const uint2*>(qrow + lane * 4);
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
      } else {
        const uint4 v = *reinterpret_cast<const uint4*>(qrow + lane * 8);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(u[i] << 16); x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
      }
      float mx = 0.f, sum = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) { mx = fmaxf(mx, fabsf(x[i])); sum += x[i]; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      constexpr int kLanesPerGroup = 64 / E;           // 16 or 8
#pragma unroll
      for (int o = kLanesPerGroup / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
      if (mx == 0.f) ex = 0;
      ex = min(max(ex, -80), 80);
      const float sf = __uint_as_float((uint32_t)(127 + 10 - ex) << 23);       // 2^(10 - ex)
      __half* dst = &sm.qh[warp][lane * E];
#pragma unroll
      for (int i = 0; i < E; ++i) dst[i] = __float2half_rn(x[i] * sf * ((i & 1) ? 0.0625f : 1.f));
      if ((lane % kLanesPerGroup) == 0) sm.qsum[warp][lane / kLanesPerGroup] = sum * P.scale_log2;
      if (lane == 0) sm.kappa[warp] = P.scale_log2 * __uint_as_float((uint32_t)(127 + 14 + ex) << 23);   // 2^(24 + ex - 10)
    }
    consumer_bar();
    uint32_t qa[8 * G][2];
    float qs[G], kap = 0.f;
    {
      const bool live = hrow < n_rep;
#pragma unroll
      for (int ks = 0; ks < 8 * G; ++ks) {
        const int gi = ks >> 2, i2 = (ks >> 1) & 1, e = ks & 1;
        const int d0 = 8 * (8 * gi + 4 * i2 + tid) + 2 * e;
        const __half* r = sm.qh[hrow];
        qa[ks][0] = live ? h2_bits(__halves2half2(r[d0], r[d0 + 4])) : 0u;
        qa[ks][1] = live ? h2_bits(__halves2half2(r[d0 + 1], r[d0 + 5])) : 0u;
      }
#pragma unroll
      for (int gi = 0; gi < G; ++gi) qs[gi] = live ? sm.qsum[hrow][gi] : 0.f;
      kap = live ? sm.kappa[hrow] : 0.f;
    }

    // ---- running state of this warp for this segment ----
    float m_run = -INFINITY, l_e = 0.f, l_o = 0.f, bias_e[Gv], bias_o[Gv];
    float o[Dv / 16][4];
#pragma unroll
    for (int i = 0; i < Gv; ++i) { bias_e[i] = 0.f; bias_o[i] = 0.f; }
#pragma unroll
    for (int i = 0; i < Dv / 16; ++i) { o[i][0] = 0.f; o[i][1] = 0.f; o[i][2] = 0.f; o[i][3] = 0.f; }
    bool poisoned = false;

    const int first = seg.c0 + (int)(((long long)warp - seg.k0 % kConsumerWarps + kConsumerWarps) % kConsumerWarps);
    for (int c = first; c < seg.c1; c += kConsumerWarps) {
      const long long k = seg.k0 + (c - seg.c0);
      const int slot = (int)(k % kSlots);
      const uint32_t round = (uint32_t)(k / kSlots);
      if (aborted || !mbar_wait(&sm.full[slot], round & 1u, &sm.abort_flag)) { aborted = true; continue; }
      if (sm.bad[slot]) {
        poisoned = true;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[slot]);
        continue;
      }
      const uint8_t* chunk = sm.ring + (size_t)slot * kChunkBytes;
      const uint4* kc4 = reinterpret_cast<const uint4*>(chunk);
      const uint4* ksb4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2));
      const uint4* vc4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2) + 128 * G);
      const uint4* vsb4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2) + 128 * G + 32 * (Dv / 2));
      const int pos0 = c * 32;
      const bool edge = pos0 < seg.lo || pos0 + 32 > seg.n;

      // ---- scores of the 4 key tiles: s2[i][e] for token 8*tid + 4*e + i, in log2 units ----
      float s2[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float acc[G][4];
#pragma unroll
        for (int gi = 0; gi < G; ++gi) { acc[gi][0] = 0.f; acc[gi][1] = 0.f; acc[gi][2] = 0.f; acc[gi][3] = 0.f; }
#pragma unroll
        for (int j = 0; j < G / 2; ++j) {
          const uint4 w4 = kc4[((i * (G / 2) + j) * 8 + g) * 4 + tid];
          const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int gi = 2 * j + (x >> 1), i2 = x & 1;
            const int ks = (gi * 2 + i2) * 2;
            const uint32_t hi = w[x] >> 8;
            mma16816(acc[gi], qa[ks][0], 0u, qa[ks][1], 0u, w[x] & kMaskLo, w[x] & kMaskHi);
            mma16816(acc[gi], qa[ks + 1][0], 0u, qa[ks + 1][1], 0u, hi & kMaskLo, hi & kMaskHi);
          }
        }
        // scale and bias of the two tokens this lane owns in tile i
        float t0 = 0.f, t1 = 0.f, u0 = 0.f, u1 = 0.f;
        if (G == 2) {
          const uint4 sb = ksb4[i * 4 + tid];
          const float2 a0 = h2_to_f2(sb.x), a1 = h2_to_f2(sb.y), b0 = h2_to_f2(sb.z), b1 = h2_to_f2(sb.w);
          t0 = acc[0][0] * a0.x; t0 = fmaf(acc[1][0], a1.x, t0);
          u0 = qs[0] * a0.y; u0 = fmaf(qs[1], a1.y, u0);
          t1 = acc[0][1] * b0.x; t1 = fmaf(acc[1][1], b1.x, t1);
          u1 = qs[0] * b0.y; u1 = fmaf(qs[1], b1.y, u1);
        } else {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const uint4 sb = ksb4[(i * 4 + tid) * 2 + e];
            const uint32_t v[4] = {sb.x, sb.y, sb.z, sb.w};
            float t = 0.f, u = 0.f;
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {
              const float2 f = h2_to_f2(v[gi]);
              t = fmaf(acc[gi][e], f.x, t);
              u = fmaf(qs[gi], f.y, u);
            }
            if (e == 0) { t0 = t; u0 = u; } else { t1 = t; u1 = u; }
          }
        }
        s2[i][0] = fmaf(kap, t0, u0);
        s2[i][1] = fmaf(kap, t1, u1);
      }
      if (edge) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int pos = pos0 + 8 * tid + 4 * e + i;
            if (pos < seg.lo || pos >= seg.n) s2[i][e] = -INFINITY;
          }
      }
      // ---- online softmax over the chunk ----
      float cm = fmaxf(fmaxf(fmaxf(s2[0][0], s2[0][1]), fmaxf(s2[1][0], s2[1][1])),
                       fmaxf(fmaxf(s2[2][0], s2[2][1]), fmaxf(s2[3][0], s2[3][1])));
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
      cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
      float m_new = fmaxf(m_run, cm);
      if (m_new == -INFINITY) m_new = 0.f;
      const float corr = fast_exp2(m_run - m_new);
      m_run = m_new;
      float p[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float off = (i & 1) ? m_new + 4.f : m_new;     // odd tiles: p / 16 (their codes carry a factor 16)
        p[i][0] = fast_exp2(s2[i][0] - off);
        p[i][1] = fast_exp2(s2[i][1] - off);
      }
      l_e = fmaf(l_e, corr, (p[0][0] + p[0][1]) + (p[2][0] + p[2][1]));
      l_o = fmaf(l_o, corr, (p[1][0] + p[1][1]) + (p[3][0] + p[3][1]));
#pragma unroll
      for (int gi = 0; gi < Gv; ++gi) { bias_e[gi] *= corr; bias_o[gi] *= corr; }
      // rescale the value accumulators when any head's running maximum moved
      if (__any_sync(0xffffffffu, corr != 1.f)) {
        const float c0 = __shfl_sync(0xffffffffu, corr, ((2 * tid) & 3) * 4);
        const float c1 = __shfl_sync(0xffffffffu, corr, ((2 * tid + 1) & 3) * 4);
#pragma unroll
        for (int mt = 0; mt < Dv / 16; ++mt) { o[mt][0] *= c0; o[mt][1] *= c1; o[mt][2] *= c0; o[mt][3] *= c1; }
      }
      // ---- p * s_v per group as two-term binary16 (rows 0..3: high part, rows 4..7: low part) ----
      uint32_t bfr[Gv][4];                                  // [group][tile] = half2(token e=0, token e=1)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float vs[2][Gv], vb[2][Gv];
        if (G == 2) {
          const uint4 sb = vsb4[i * 4 + tid];
          const float2 a0 = h2_to_f2(sb.x), a1 = h2_to_f2(sb.y), b0 = h2_to_f2(sb.z), b1 = h2_to_f2(sb.w);
          vs[0][0] = a0.x; vb[0][0] = a0.y; vs[0][1] = a1.x; vb[0][1] = a1.y;
          vs[1][0] = b0.x; vb[1][0] = b0.y; vs[1][1] = b1.x; vb[1][1] = b1.y;
        } else {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const uint4 sb = vsb4[(i * 4 + tid) * 2 + e];
            const uint32_t v[4] = {sb.x, sb.y, sb.z, sb.w};
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) { const float2 f = h2_to_f2(v[gi]); vs[e][gi] = f.x; vb[e][gi] = f.y; }
          }
        }
        if (edge) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int pos = pos0 + 8 * tid + 4 * e + i;
            if (pos < seg.lo || pos >= seg.n) {
#pragma unroll
              for (int gi = 0; gi < Gv; ++gi) { vs[e][gi] = 0.f; vb[e][gi] = 0.f; }
            }
          }
        }
#pragma unroll
        for (int gi = 0; gi < Gv; ++gi) {
          const float x0 = p[i][0] * vs[0][gi], x1 = p[i][1] * vs[1][gi];
          const __half2 h = __floats2half2_rn(x0, x1);
          const float r0 = fmaf(-delta, __low2float(h), x0), r1 = fmaf(-delta, __high2float(h), x1);
          bfr[gi][i] = h2_bits(__floats2half2_rn(r0, r1));
          if (i & 1) bias_o[gi] = fmaf(p[i][0], vb[0][gi], fmaf(p[i][1], vb[1][gi], bias_o[gi]));
          else bias_e[gi] = fmaf(p[i][0], vb[0][gi], fmaf(p[i][1], vb[1][gi], bias_e[gi]));
        }
      }
      // ---- P.V on the codes: 16 value rows x 8 columns (heads hi|lo) x 32 tokens per tile pair ----
#pragma unroll
      for (int q4 = 0; q4 < Dv / 32; ++q4) {
        const uint4 w4 = vc4[(q4 * 8 + g) * 4 + tid];
        const int gi = q4 >> 1;
        {
          const uint32_t xh = w4.x >> 8, yh = w4.y >> 8;
          mma16816(o[2 * q4], w4.x & kMaskLo, w4.y & kMaskLo, w4.x & kMaskHi, w4.y & kMaskHi, bfr[gi][0], bfr[gi][1]);
          mma16816(o[2 * q4], xh & kMaskLo, yh & kMaskLo, xh & kMaskHi, yh & kMaskHi, bfr[gi][2], bfr[gi][3]);
        }
        {
          const uint32_t xh = w4.z >> 8, yh = w4.w >> 8;
          mma16816(o[2 * q4 + 1], w4.z & kMaskLo, w4.w & kMaskLo, w4.z & kMaskHi, w4.w & kMaskHi, bfr[gi][0], bfr[gi][1]);
          mma16816(o[2 * q4 + 1], xh & kMaskLo, yh & kMaskLo, xh & kMaskHi, yh & kMaskHi, bfr[gi][2], bfr[gi][3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot]);
    }

    // ---- flush this warp's state to shared memory ----
    {
      float l = l_e + 16.f * l_o;
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
      float bias[Gv];
#pragma unroll
      for (int gi = 0; gi < Gv; ++gi) {
        float b = bias_e[gi] + 16.f * bias_o[gi];
        b += __shfl_xor_sync(0xffffffffu, b, 1);
        b += __shfl_xor_sync(0xffffffffu, b, 2);
        bias[gi] = b;
      }
      float (*mg)[S::kMergeStride] = sm.merge[warp];
      if (g < 4 && tid == 0) {
        mg[g][Dv] = m_run;
        mg[g][Dv + 1] = (poisoned || aborted) ? -1.f : l;
#pragma unroll
        for (int gi = 0; gi < Gv; ++gi) mg[g][Dv + 2 + gi] = bias[gi];
      }
      // columns 4..7 (lanes tid 2,3) hold the low-part products of heads 0..3
#pragma unroll
      for (int mt = 0; mt < Dv / 16; ++mt) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float v = o[mt][r] + __shfl_xor_sync(0xffffffffu, o[mt][r], 2);
          if (tid < 2) mg[2 * tid + (r & 1)][16 * mt + g + 8 * (r >> 1)] = v * 16777216.f;
        }
      }
    }
    consumer_bar();
    // ---- combine the four warps, write the segment's partial record ----
    {
      const int pair = seg.a * y.Hkv + seg.hk;
      float* rec = P.partials + (size_t)(pair + cta) * n_rep * (Dv + 2);
      const int t = threadIdx.x;
      for (int idx = t; idx < n_rep * Dv; idx += kConsumerThreads) {
        const int h = idx / Dv, d = idx % Dv, gi = d >> 6;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, sm.merge[w][h][Dv]);
        float a = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
          const float mw = sm.merge[w][h][Dv];
          if (mw != -INFINITY) a += exp2f(mw - M) * (sm.merge[w][h][d] + sm.merge[w][h][Dv + 2 + gi]);
        }
        rec[(size_t)h * (Dv + 2) + d] = a;
      }
      if (t < n_rep) {
        const int h = t;
        float M = -INFINITY, Lsum = 0.f;
        bool bad = false;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, sm.merge[w][h][Dv]);
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
          const float mw = sm.merge[w][h][Dv], lw = sm.merge[w][h][Dv + 1];
          if (lw < 0.f) bad = true;
          if (mw != -INFINITY) Lsum += exp2f(mw - M) * lw;
        }
        rec[(size_t)h * (Dv + 2) + Dv] = M;
        rec[(size_t)h * (Dv + 2) + Dv + 1] = bad ? -1.f : Lsum;
      }
      if (seg.first_of_pair && t == 0) {
        bool bad;
        const AgentRange r = agent_range(P.kv_lens, seg.a, P.window, P.max_blocks, bad);
        const long long pair_last = seg.u0 + (r.cf + r.nc - seg.c0) - 1;
        P.desc[pair] = make_int2(cta, cta_of_unit(U, pair_last, n_ctas));
      }
    }
    consumer_bar();
  }
  if (aborted && lane == 0) raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
}

// grid: (Hkv, A); combines the partial records of one (agent, KV head) pair and writes n_rep output rows
__global__ void __launch_bounds__(128)
decode_mma_merge_kernel(Layout y, int n_agents, int max_blocks, const int32_t* __restrict__ kv_lens, int window,
                        const int2* __restrict__ desc, const float* __restrict__ partials, void* __restrict__ out,
                        int out_dtype, float* __restrict__ lse) {
  const int hk = blockIdx.x, a = blockIdx.y;
  const int Dv = y.Dv, n_rep = y.n_rep;
  bool bad_len;
  const AgentRange r = agent_range(kv_lens, a, window, max_blocks, bad_len);
  const int pair = a * y.Hkv + hk;
  int c_first = 0, c_last = -1;
  if (r.nc > 0) { const int2 d = desc[pair]; c_first = d.x; c_last = d.y; }
  for (int h = 0; h < n_rep; ++h) {
    float M = -INFINITY;
    for (int c = c_first; c <= c_last; ++c)
      M = fmaxf(M, partials[((size_t)(pair + c) * n_rep + h) * (Dv + 2) + Dv]);
    float Lsum = 0.f;
    bool poisoned = false;
    for (int c = c_first; c <= c_last; ++c) {
      const float* rec = partials + ((size_t)(pair + c) * n_rep + h) * (Dv + 2);
      if (rec[Dv + 1] < 0.f) poisoned = true;
      if (rec[Dv] != -INFINITY) Lsum += exp2f(rec[Dv] - M) * rec[Dv + 1];
    }
    if (poisoned) Lsum = 0.f;
    const size_t row = (size_t)a * y.Hq + (size_t)hk * n_rep + h;
    for (int d = threadIdx.x; d < Dv; d += blockDim.x) {
      float acc = 0.f;
      for (int c = c_first; c <= c_last; ++c) {
        const float* rec = partials + ((size_t)(pair + c) * n_rep + h) * (Dv + 2);
        if (rec[Dv] != -INFINITY) acc += exp2f(rec[Dv] - M) * rec[d];
      }
      const float v = Lsum > 0.f ? acc / Lsum : 0.f;
      if (out_dtype == Q4KV_OUT_BF16) reinterpret_cast<__nv_bfloat16*>(out)[row * Dv + d] = __float2bfloat16_rn(v);
      else reinterpret_cast<float*>(out)[row * Dv + d] = v;
    }
    if (threadIdx.x == 0 && lse) lse[row] = Lsum > 0.f ? (M + log2f(Lsum)) / kLog2e : -INFINITY;
  }
}

int decode_grid(const Layout& y, int n_agents, int max_kv_len) {
  const long long units = (long long)n_agents * y.Hkv * ((max_kv_len + 31) / 32 + 1);
  const long long cap = 148 * kCtasPerSm;
  return (int)(units < cap ? (units < 1 ? 1 : units) : cap);
}

template <int G>
cudaError_t launch_g(const DecodeParams& P, int grid, cudaStream_t st) {
  const size_t smem = sizeof(Smem<G>);
  cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  decode_mma_kernel<G><<<grid, kThreads, smem, st>>>(P);
  return cudaGetLastError();
}

}  // namespace

bool decode_mma_supported(const Layout& y) {
  return !y.alias && y.D == y.Dv && (y.D == 128 || y.D == 256) && y.n_rep <= 4;
}

size_t decode_mma_workspace_bytes(const Layout& y, int n_agents) {
  const size_t pairs = (size_t)n_agents * y.Hkv;
  const size_t desc = (pairs * sizeof(int2) + 255) & ~(size_t)255;
  return desc + (pairs + 148 * kCtasPerSm) * y.n_rep * (y.Dv + 2) * sizeof(float);
}

cudaError_t launch_decode_mma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                              const int32_t* kv_lens, int max_kv_len, int window, const void* q, float scale,
                              void* out, int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st) {
  if (b.n_agents <= 0) return cudaSuccess;
  const size_t pairs = (size_t)b.n_agents * y.Hkv;
  const size_t desc_bytes = (pairs * sizeof(int2) + 255) & ~(size_t)255;
  DecodeParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents;
  P.max_blocks = b.max_blocks; P.tables = b.block_tables; P.kv_lens = kv_lens; P.window = window;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e;
  P.desc = (int2*)ws; P.partials = (float*)((uint8_t*)ws + desc_bytes); P.flags = flags;
  const int span = (window > 0 && window + 32 < max_kv_len) ? window + 32 : max_kv_len;
  const int grid = decode_grid(y, b.n_agents, span);
  cudaError_t e = y.G == 2 ? launch_g<2>(P, grid, st) : launch_g<4>(P, grid, st);
  if (e != cudaSuccess) return e;
  dim3 mgrid(y.Hkv, b.n_agents);
  decode_mma_merge_kernel<<<mgrid, 128, 0, st>>>(y, b.n_agents, b.max_blocks, kv_lens, window, P.desc, P.partials, out,
                                                 out_dtype, lse);
  return cudaGetLastError();
}

}  // namespace q4kv
