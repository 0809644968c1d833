// q4kv_decode_attention, tensor-core path for GQA shapes (d_qk = d_v in {128, 256}, at most four
// query heads per KV head): one query token per agent over its whole Q4 cache, read in place
// (Section 3.4 "Batched Quantized Inference": fused attention on the Q4 tensors; Section 3.6:
// GQA head mapping and sliding-window layers).
//
// The kernel is bound by HBM bandwidth, so it is organised around the byte stream:
//   * Work = the flattened list of 32-token chunks of all (agent, KV head) pairs inside their key
//     range [lo, kv_len).  The list is cut into equal contiguous ranges, one per persistent CTA
//     (one CTA per SM), so ragged lengths balance by construction.  A CTA's range may cover
//     parts of several pairs ("segments").  A pair that lies inside one CTA is finished there;
//     otherwise every CTA that holds a piece writes a partial (m, l, acc) record and takes a
//     ticket, and the CTA that draws the last ticket combines the records -- one launch, no
//     waiting on other CTAs.
//   * The CTA's chunks stream through a shared-memory ring with one bulk asynchronous copy per
//     chunk (a chunk is one contiguous byte range of the pool) completing on an mbarrier.  A
//     planner warp walks the CTA's range ahead of the copies, 32 chunks per step in lockstep, and
//     leaves each chunk's pool offset in a small shared-memory table; between steps it polls the
//     ring, one lane per slot but all lanes on one path, and issues the copy of the next chunk of
//     every slot whose previous chunk has been consumed.  The
//     consumer warps run independently of one another: each claims the next chunk from a shared
//     counter, keeps its own online-softmax state, and on leaving a segment deposits that state in
//     shared memory; the warp that makes the deposit count complete combines the deposits and does
//     the segment's epilogue (output, or record + ticket) while the others are already working on
//     the next segment.  No CTA-wide barrier after start-up.
//   * Arithmetic runs on the 4-bit codes, not on dequantized values.  With x^ = c*s + b and one
//     (s, b) per token and 64-element group,
//         q.k_t   = sum_g [ s_tg * (sum_{d in g} q_d c_td) + b_tg * (sum_{d in g} q_d) ]
//         (p.V)_d = sum_t (p_t s_tg(d)) c_td + sum_t p_t b_tg(d).
//     Both contractions are mma.sync m16n8k16 f16 with the code operand produced by masking the
//     packed word in place: a nibble in the low bits of a 16-bit lane IS the binary16 subnormal
//     c * 2^-24, and one nibble up it is 16c * 2^-24 -- the 16 is divided out of the other operand
//     (the matching query elements for q.K, the probabilities of odd key tiles for p.V).  The bf16
//     query is scaled per row by a power of two into binary16, so nothing is rounded before the
//     products, which are exact.  (The 8-bit float forms of mma.sync are not used: on this part
//     each costs two f16 tensor instructions plus conversions and adds.)
//   * In the score product the key codes are the A operand (16 tokens x 16 head-dim elements) and the
//     query the B operand (eight columns: the query heads 0..3 and their repeats), so a KV head's
//     codes are unpacked once for all its query heads.  The probabilities times the token's value
//     scale are transposed across the warp (movmatrix) into the B operand of the value product,
//     whose A operand is the token-packed value words.  Columns 4..7 carry the low half of a
//     two-term binary16 split of p*s, which makes the value product accurate to ~2^-22 at no
//     extra MMA.
#include <climits>

#include "q4kv_layout.cuh"
#include "quantize_core.cuh"

namespace q4kv {

namespace {

constexpr int kMaxGrid = 512;                          // upper bound on the persistent grid (one CTA per SM)
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
__device__ inline bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_test_wait(bar, parity)) return true;        // the usual case: the chunk landed long ago (a blocking try costs more)
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// Bounded spin on a shared-memory word until it reaches `want`.
__device__ inline bool spin_until_ge(volatile int* word, int want, volatile int* abort_flag) {
  for (uint32_t i = 0; i < (kSpinLimit << 4); ++i) {
    if (*word >= want) return true;
#ifdef Q4KV_SPIN_SLEEP
    __nanosleep(Q4KV_SPIN_SLEEP);
#endif
    if ((i & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ inline void prefetch_l2_bulk(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ inline void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ inline void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ inline void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ inline void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ inline float fast_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
// half2(lo = a, hi = b), both rounded toward zero
__device__ inline uint32_t f32x2_to_h2_rz(float a, float b) {
  uint32_t r;
  asm("cvt.rz.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
  return r;
}
__device__ inline uint32_t f32x2_to_h2_rn(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

constexpr int kMaxLayersPerCall = 64;
struct DecodeParams {
  Layout y;
  const uint8_t* pool;
  int n_blocks, layer, n_agents, max_blocks, len_cap;
  // Several layers in one launch (the layer-batched entry): the work list runs over "virtual agents" v = li * n_real + a
  // (layer li of the call, real agent a).  q, out, lse, the new rows, the arrival counters and the partial records are
  // all indexed by v; lengths and block tables by a; the window and the pool layer by li.  n_agents = layer_count * n_real.
  int n_real, layer_count;
  int windows[kMaxLayersPerCall];   // sliding window of each layer of the call (0: none)
  const int32_t* tables;
  const int32_t* kv_lens;
  const uint16_t* q;          // bf16 [layer_count][A][Hq][D]
  float scale_log2;           // softmax_scale * log2(e)
  int32_t* tickets;           // [A*Hkv], zero between calls
  float* partials;            // [A*Hkv + grid][n_rep][Dv + 4]
  void* out;
  int out_dtype;
  float* lse;
  int32_t* flags;
  const uint16_t* k_new;      // fused append: bf16 [A][Hkv][D] rows of the token at position kv_len - 1 (null: none)
  const uint16_t* v_new;
};

// ---------------------------------------------------------------------------------------------
// Work list: chunks of all (agent, KV head) pairs, agent-major, then head, then chunk
// ---------------------------------------------------------------------------------------------
struct AgentRange { int n, lo, cf, nc; };   // keys [lo, n); chunks cf .. cf+nc-1

// len_cap: the host's bound on every length (at most max_blocks * 256); longer or negative lengths are rejected
__device__ inline AgentRange agent_range(const DecodeParams& P, int a, bool& bad) {
  AgentRange r;
  const int li = P.layer_count > 1 ? a / P.n_real : 0;
  const int window = P.windows[li];
  r.n = P.kv_lens[a - li * P.n_real];
  bad = r.n < 0 || r.n > P.len_cap;
  if (bad) r.n = 0;
  r.lo = window > 0 ? max(0, r.n - window) : 0;
  r.cf = r.lo >> 5;
  r.nc = r.n > r.lo ? ((r.n + 31) >> 5) - r.cf : 0;
  return r;
}

// Equal partition of U units over n CTAs (all quantities fit 31 bits; the host checks):
// the first U % n CTAs own U / n + 1 units, the others U / n.  Requires n <= U.
struct Partition {
  uint32_t U, n, q, r;
  __device__ void init(uint32_t U_, uint32_t n_) { U = U_; n = n_; q = U_ / n_; r = U_ - q * n_; }
  __device__ uint32_t begin(uint32_t c) const { return c * q + (c < r ? c : r); }
  __device__ int cta_of(uint32_t u) const {
    const uint32_t big = r * (q + 1);
    return u < big ? (int)(u / (q + 1)) : (int)(r + (u - big) / q);
  }
};

// Warp-cooperative: total number of units U, this CTA's range and the agent that contains its
// first unit.  One pass over the agents when there are at most 32 of them.
struct RangeStart { uint32_t U, u_begin, u_end, agent_start; int n_ctas, agent; bool any_bad; Partition part; };

__device__ inline RangeStart find_range(const DecodeParams& P, int cta, int grid) {
  const int lane = threadIdx.x & 31;
  const int n_agents = P.n_agents, Hkv = P.y.Hkv;
  RangeStart rs;
  rs.any_bad = false;
  rs.agent = -1;
  rs.agent_start = 0;
  uint32_t cum = 0, inc0 = 0, cnt0 = 0;
  for (int base = 0; base < n_agents; base += 32) {
    const int a = base + lane;
    uint32_t cnt = 0;
    bool bad = false;
    if (a < n_agents) cnt = (uint32_t)(agent_range(P, a, bad).nc * Hkv);
    rs.any_bad |= __any_sync(0xffffffffu, bad);
    uint32_t inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (base == 0) { inc0 = inc; cnt0 = cnt; }
    cum += __shfl_sync(0xffffffffu, inc, 31);
  }
  rs.U = cum;
  rs.n_ctas = (uint32_t)grid < cum ? grid : (int)cum;
  rs.u_begin = rs.u_end = 0;
  rs.part.U = 0; rs.part.n = 1; rs.part.q = 0; rs.part.r = 0;
  if (cum == 0 || cta >= rs.n_ctas) return rs;
  rs.part.init(cum, (uint32_t)rs.n_ctas);
  rs.u_begin = rs.part.begin(cta);
  rs.u_end = rs.part.begin(cta + 1);
  const uint32_t want = rs.u_begin;
  if (n_agents <= 32) {
    const unsigned bal = __ballot_sync(0xffffffffu, inc0 > want);
    const int l = __ffs(bal) - 1;
    rs.agent = l;
    rs.agent_start = __shfl_sync(0xffffffffu, inc0, l) - __shfl_sync(0xffffffffu, cnt0, l);
    return rs;
  }
  cum = 0;
  for (int base = 0; base < n_agents; base += 32) {
    const int a = base + lane;
    uint32_t cnt = 0;
    bool bad = false;
    if (a < n_agents) cnt = (uint32_t)(agent_range(P, a, bad).nc * Hkv);
    uint32_t inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const uint32_t tot = __shfl_sync(0xffffffffu, inc, 31);
    if (want < cum + tot) {
      const unsigned bal = __ballot_sync(0xffffffffu, cum + inc > want);
      const int l = __ffs(bal) - 1;
      rs.agent = base + l;
      rs.agent_start = cum + __shfl_sync(0xffffffffu, inc, l) - __shfl_sync(0xffffffffu, cnt, l);
      return rs;
    }
    cum += tot;
  }
  return rs;
}

// One segment: the part of pair (agent a, KV head hk) inside this CTA's unit range.  A segment is walked from its last
// chunk to its first (the order does not matter to the online softmax).  With the fused append, the chunk of the agent's
// newest position -- the pair's last chunk -- is patched by the planner warp after it has landed; it is moved a few
// places back in the walk (to place tail_pos), so that the consumers have other chunks to work on meanwhile.
constexpr int kTailPos = 14;
struct Segment {
  int a, hk, c0, c1;      // (virtual) agent, KV head, logical chunk indices [c0, c1) of the agent
  int ar, li;             // real agent (lengths, block table) and layer of the call (pool layer)
  int n, lo;              // key range of the agent
  int cf, nc;             // the pair's whole chunk range
  int k0;                 // running chunk counter of the CTA at c0
  uint32_t u0;            // global unit index at c0
  int tail_pos;           // place in the walk of the chunk that receives the new token; -1: none in this segment
  __device__ void set_tail(bool fused) {
    const int cnt = c1 - c0;
    tail_pos = (fused && c1 == cf + nc) ? (cnt - 1 < kTailPos ? cnt - 1 : kTailPos) : -1;
  }
  __device__ int chunk_at(int j) const {    // logical chunk at place j of the walk, 0 <= j < c1 - c0
    if (tail_pos < 0 || j > tail_pos) return c1 - 1 - j;
    return j == tail_pos ? c1 - 1 : c1 - 2 - j;
  }
};

struct Walker {
  const DecodeParams* P;
  int n_agents, Hkv;
  uint32_t u, u_end;
  int k, a, hk, c;
  bool fused;               // the launch appends one token per agent
  AgentRange r;

  __device__ void init(const DecodeParams& P_, const RangeStart& rs) {
    P = &P_; n_agents = P_.n_agents; Hkv = P_.y.Hkv; fused = P_.k_new != nullptr;
    u = rs.u_begin; u_end = rs.u_end; k = 0;
    a = rs.agent; hk = 0; c = 0;
    r.n = 0; r.lo = 0; r.cf = 0; r.nc = 0;
    if (u < u_end && a >= 0) {
      bool bad;
      r = agent_range(*P, a, bad);
      const uint32_t rem = u - rs.agent_start;
      hk = (int)(rem / (uint32_t)r.nc);
      c = r.cf + (int)(rem - (uint32_t)hk * (uint32_t)r.nc);
    }
  }
  __device__ bool next(Segment& s) {
    if (u >= u_end || a < 0) return false;
    const int pair_end = r.cf + r.nc;
    const uint32_t left = u_end - u;
    const int c1 = (uint32_t)(pair_end - c) <= left ? pair_end : c + (int)left;
    s.li = P->layer_count > 1 ? a / P->n_real : 0; s.ar = a - s.li * P->n_real;
    s.a = a; s.hk = hk; s.c0 = c; s.c1 = c1; s.n = r.n; s.lo = r.lo; s.cf = r.cf; s.nc = r.nc; s.k0 = k; s.u0 = u;
    s.set_tail(fused);
    const int cnt = c1 - c;
    u += (uint32_t)cnt; k += cnt;
    if (c1 == pair_end) {
      ++hk;
      if (hk == Hkv) {
        hk = 0;
        bool bad;
        do {
          ++a;
          if (a >= n_agents) { a = -1; break; }
          r = agent_range(*P, a, bad);
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

__host__ __device__ constexpr int kRecStride(int Dv) { return Dv + 4; }
// The kernel is instantiated by the number of key groups G: 2 and 4 are the symmetric shapes (d_qk = d_v = 64 G), 3 is
// the asymmetric per-head MLA cache of Section 3.6 (d_qk 192, d_v 128).
__host__ __device__ constexpr int value_groups(int G) { return G == 3 ? 2 : G; }   // acc[Dv], m, l, pad: 16-byte multiples
constexpr int kQBufs = 4;      // query-fragment buffers (segments s, s+4, ... share one)
constexpr int kOffCap = 256;   // entries of the planner's offset table (a ring over the CTA's chunk indices)
constexpr int kTailQ = 8;      // chunks waiting for the planner's patch (planning stops while the queue is full)
constexpr uint32_t kOffBad = 0xFFFFFFFFu;   // table entry of a chunk whose block id is outside the pool
constexpr int kSmemBudget = 232448 - 2048;   // 227 KB per CTA, less the small arrays of the structure below

// consumer warps per CTA.  Two warps per scheduler: the hot loop wants ~180 registers per thread at d = 128 and ~245 at
// d = 256, and with three warps per scheduler (168 registers) what the compiler moves to local memory costs more than
// the third warp brings, since almost no L1 is left beside the ring (measured: 78 against 71 us on 40 agents x 4096)
#ifndef Q4KV_DECODE_WARPS_D128
#define Q4KV_DECODE_WARPS_D128 7
#endif
#ifndef Q4KV_DECODE_WARPS_D256
#define Q4KV_DECODE_WARPS_D256 7
#endif

template <int G, int NW>
struct Smem {
  static constexpr int D = 64 * G, Gv = value_groups(G), Dv = 64 * Gv;
  static constexpr int kChunkBytes = 32 * (D / 2 + 4 * G + Dv / 2 + 4 * Gv);
  static constexpr int kMergeStride = Dv + 8;           // acc[Dv], m, l, bias[Gv], pad
  // deposit buffers (consecutive segments alternate).  One at d = 256: its 30 KB are worth more as four ring slots (20
  // instead of 16: the global layer of the ragged benchmark runs 1.2 % faster, bytes in flight being what limits it)
  static constexpr int kMBufs = G == 4 ? 1 : 2;
  static constexpr int kRingBudget = kSmemBudget - kMBufs * NW * 4 * kMergeStride * 4 - kQBufs * 2 * G * 32 * 16;
  static constexpr int kSlots = kRingBudget / kChunkBytes < 32 ? kRingBudget / kChunkBytes : 32;   // one producer lane per slot
  alignas(128) uint8_t ring[kSlots * kChunkBytes];
  alignas(16) float merge[kMBufs][NW][4][kMergeStride];
  alignas(16) uint4 qfrag[kQBufs][2 * G][32];           // [buffer][key word of a lane][lane = row * 4 + tid] = A registers
  float qsum[kQBufs][4][G];                             // scale_log2 * sum of the true q over each group
  float kappa[kQBufs][4];                               // scale_log2 * 2^(ex + 13)
  alignas(8) uint64_t full[kSlots];
  uint32_t src_off[kOffCap];    // pool offset (16-byte units inside the layer) of chunk k at k % kOffCap; kOffBad: bad block id
  int released[kSlots];         // number of times each slot has been consumed (monotonic: no parity aliasing)
  int patched[kSlots];          // round + 1 of the last chunk the planner has patched in each slot (fused append)
  int4 tail_q[kTailQ];          // planner's queue of chunks to patch: (chunk index in the CTA, agent, KV head, token in chunk)
  int bad[kSlots];
  int q_tag[kQBufs];            // s + 1 once the query of segment s is staged in buffer s % kQBufs
  int deposits[kMBufs];         // running count of deposits into each buffer
  int epilogues[kMBufs];        // number of completed epilogues of each buffer
  int next_chunk;               // claim counter
  int epi_claim[kMBufs];        // uses of each deposit buffer whose epilogue has been taken (by a consumer or the planner)
  int all_issued;               // set by the planner once every chunk of the CTA has been issued
  int fin_arrived;              // last segment: head warps whose record is written
  int fin_ticket;               // last segment: 0 until the ticket is drawn, then 1 (not the last) or 2 (combine the records)
  int abort_flag;
};

// Online-softmax state of one warp for one segment.  A lane owns two score columns (2 * tid, 2 * tid + 1 of eight:
// columns 0..3 are the query heads, 4..7 repeat them) and, of every 32-token chunk, the four tokens 4 * g .. 4 * g + 3;
// m, l and the bias sums are per column, partial over the lane's tokens.
template <int G>
struct WarpState {
  static constexpr int Gv = value_groups(G);
  float m[2], l_e[2], l_o[2], bias_e[2][Gv], bias_o[2][Gv];
  float o[4 * Gv][4];
  __device__ void reset() {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      m[c] = -INFINITY; l_e[c] = 0.f; l_o[c] = 0.f;
#pragma unroll
      for (int i = 0; i < Gv; ++i) { bias_e[c][i] = 0.f; bias_o[c][i] = 0.f; }
    }
#pragma unroll
    for (int i = 0; i < 4 * Gv; ++i) { o[i][0] = 0.f; o[i][1] = 0.f; o[i][2] = 0.f; o[i][3] = 0.f; }
  }
};

// Warp-level: stage the query rows of one pair as binary16 in A-fragment order (each row scaled by a
// power of two, so nothing is rounded), plus the per-group sums of the true query and the per-head
// factor that undoes the scaling.  Key word w = 8*gi + 4*i2 + t of a token holds elements 8w..8w+7
// and feeds two 16x8x16 products: (0,4 | 1,5) and (2,6 | 3,7), where the second pair of each meets
// codes in nibble 1 of their 16-bit lanes (a factor 16, divided out of the query here).  The uint4
// of word p = 2*gi + i2 is {a0, a2} of the first product and {a0, a2} of the second, for the lane
// (row h, t); rows h + 4 repeat rows h, so that lanes g and g + 4 see the same scores.
template <int G>
__device__ __noinline__ void stage_query(uint4 (*qfrag)[32], float (*qsum)[G], float* kappa,
                                         const uint16_t* __restrict__ q, int Hq, int n_rep, float scale_log2, int a,
                                         int hk, int lane) {
  constexpr int D = 64 * G;
  // a row's D / 8 words sit in kRowLanes consecutive lanes (a power of two, so that the row maximum is a butterfly)
  constexpr int kRowLanes = D / 8 <= 16 ? 16 : 32;
  for (int base = 0; base < n_rep * kRowLanes; base += 32) {
    const int idx = base + lane;
    const int h_raw = idx / kRowLanes, w = idx % kRowLanes;
    const bool valid = h_raw < n_rep && w < D / 8;
    const int h = valid ? h_raw : 0;
    const uint16_t* qrow = q + ((size_t)a * Hq + (size_t)hk * n_rep + h) * D;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (valid) v = *reinterpret_cast<const uint4*>(qrow + 8 * w);
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(u[i] << 16); x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
    // row maximum and group sums: the D/8 lanes of a row are consecutive (16 or 32)
    float mx = 0.f, sum = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { mx = fmaxf(mx, fabsf(x[i])); sum += x[i]; }
#pragma unroll
    for (int o = kRowLanes / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);   // 8 words per group
    if (!valid) continue;
    int ex = (int)((__float_as_uint(mx) >> 23) & 255u) - 127;
    if (mx == 0.f) ex = 0;
    ex = min(max(ex, -100), 100);
    const float sf = __uint_as_float((uint32_t)(127 + 11 - ex) << 23);         // 2048 <= max |q| * sf < 4096
    const float sl = sf * 0.0625f;
    const uint4 f = make_uint4(f32x2_to_h2_rn(x[0] * sf, x[4] * sf), f32x2_to_h2_rn(x[1] * sl, x[5] * sl),
                               f32x2_to_h2_rn(x[2] * sf, x[6] * sf), f32x2_to_h2_rn(x[3] * sl, x[7] * sl));
    const int gi = w >> 3, i2 = (w >> 2) & 1, t = w & 3;
    qfrag[2 * gi + i2][h * 4 + t] = f;
    qfrag[2 * gi + i2][(h + 4) * 4 + t] = f;
    if ((w & 7) == 0) qsum[h][gi] = sum * scale_log2;
    if (w == 0) kappa[h] = scale_log2 * __uint_as_float((uint32_t)(127 + 13 + ex) << 23);  // 2^24 / sf
  }
}

// Fused append (one new token per agent): the planner warp of the CTA that holds the chunk of an agent's newest position
// quantizes that token's K and V rows (Section 3.2 quantizer, the same device function the append kernel uses) and
// writes them into the chunk once it has landed -- in shared memory for this launch, in the pool for the following
// ones -- and then lets the chunk's consumer go on.  Every chunk is held by exactly one CTA of the grid, so nobody else
// reads or writes these words during the launch.
// Eight consecutive lanes own one 64-element group; the 8-lane shuffles never straddle K and V (D / 8 is a multiple
// of 8).  The value codes are token-packed: one nibble of each of the row's d_v words is replaced.
template <int G>
__device__ __noinline__ void append_new_token(uint8_t* chunk, uint8_t* gchunk, const Layout& y,
                                              const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                                              int a, int hk, int tau, int lane) {
  constexpr int D = 64 * G, Gv = value_groups(G), Dv = 64 * Gv, W = D / 8, Wv = Dv / 8;   // words per K row, per V row
  const size_t head = (size_t)a * y.Hkv + hk;
#pragma unroll
  for (int base = 0; base < W + Wv; base += 32) {
    const int idx = base + lane;
    const bool live = idx < W + Wv;                      // W + Wv need not be a multiple of 32: idle lanes quantize zeros
    const bool is_v = idx >= W;
    const int w = is_v ? (idx - W) % Wv : idx;
    float x[8];
    {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (live) v = *reinterpret_cast<const uint4*>(is_v ? v_new + head * Dv + 8 * w : k_new + head * D + 8 * w);
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) { x[2 * i] = __uint_as_float(u[i] << 16); x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
    }
    const QuantOut qo = quantize_eight(x, y.sb_bf16 != 0);
    const uint32_t sb = qo.sb;
    if (!live) continue;
    if (!is_v) {
      const uint32_t at = y.off_kc + 4u * k_word_offset(tau, w, G);
      *reinterpret_cast<uint32_t*>(chunk + at) = qo.word;
      *reinterpret_cast<uint32_t*>(gchunk + at) = qo.word;
      if ((w & 7) == 0) {
        const uint32_t sat = y.off_ksb + 4u * sb_offset(tau, w >> 3, G);
        *reinterpret_cast<uint32_t*>(chunk + sat) = sb;
        *reinterpret_cast<uint32_t*>(gchunk + sat) = sb;
      }
    } else {
      const int shift = 4 * (tau & 7);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t at = y.off_vc + 4u * v_word_offset(tau >> 3, 8 * w + e);
        const uint32_t old = *reinterpret_cast<const uint32_t*>(chunk + at);
        const uint32_t nw = (old & ~(0xFu << shift)) | (((qo.word >> (4 * e)) & 0xFu) << shift);
        *reinterpret_cast<uint32_t*>(chunk + at) = nw;
        *reinterpret_cast<uint32_t*>(gchunk + at) = nw;
      }
      if ((w & 7) == 0) {
        const uint32_t sat = y.off_vsb + 4u * sb_offset(tau, w >> 3, Gv);
        *reinterpret_cast<uint32_t*>(chunk + sat) = sb;
        *reinterpret_cast<uint32_t*>(gchunk + sat) = sb;
      }
    }
  }
  __syncwarp();                                          // the patched chunk is read by the same warp
}

// Ask for the new token's rows early (when the segment's query is staged), so that the warp that later owns the
// chunk finds them in L2.
template <int G>
__device__ inline void prefetch_new_token(const uint16_t* k_new, const uint16_t* v_new, int Hkv, int a, int hk, int lane) {
  constexpr int D = 64 * G, Dv = 64 * value_groups(G), kLines = D * 2 / 128, kLinesV = Dv * 2 / 128;   // 128-byte lines per row
  if (lane < kLines + kLinesV) {
    const size_t head = (size_t)a * Hkv + hk;
    const uint16_t* p = lane < kLines ? k_new + head * D + lane * 64 : v_new + head * Dv + (lane - kLines) * 64;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
  }
}

// Transpose of an 8 x 8 matrix of 16-bit elements held one row per lane group (lane l: row l / 4, columns 2 * (l % 4)
// and + 1): afterwards lane l holds row l / 4 of the transposed matrix.
__device__ inline uint32_t transpose_8x8_b16(uint32_t a) {
  uint32_t d;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// One 32-token chunk against this warp's query fragments.
//   Scores: the key codes are the A operand (16 tokens x 16 head-dim elements per product: lane (g, tid) holds the words
//   of the tokens 4g + i, i = 0..3, so products pair the token rows (0, 1) and (2, 3)), the query the B operand (eight
//   columns: heads 0..3 and their repeats).  A lane ends up with the scores of its four tokens for columns 2 tid and
//   2 tid + 1.  The probabilities, multiplied by the token's value scale, are packed two columns to a register and
//   transposed across the warp (movmatrix) into the B operand of the value product, whose A operand is the token-packed
//   value words; columns 4..7 carry the low half of the two-term split of p * s.
template <int G, bool kBf>
__device__ __forceinline__ void process_chunk(const uint8_t* chunk, int pos0, int key_lo, int key_n, int g, int tid,
                                              const uint4* qb, const float (&qs)[2][G], const float (&kap)[2],
                                              uint32_t split_mask, WarpState<G>& st) {
  constexpr int D = 64 * G, Gv = value_groups(G), Dv = 64 * Gv;
  const uint4* kc4 = reinterpret_cast<const uint4*>(chunk);
  const uint8_t* ksb = chunk + 32 * (D / 2);
  const uint4* vc4 = reinterpret_cast<const uint4*>(chunk + 32 * (D / 2) + 128 * G);
  const uint8_t* vsb = chunk + 32 * (D / 2) + 128 * G + 32 * (Dv / 2);
  const bool edge = pos0 < key_lo || pos0 + 32 > key_n;

  // ---- scores sc[i][c] of token 4g + i for column 2 tid + c, in log2 units ----
  float sc[4][2];
  {
    float acc[2][G][4];                                  // [token-row pair][group]
#pragma unroll
    for (int pr = 0; pr < 2; ++pr)
#pragma unroll
      for (int gi = 0; gi < G; ++gi) { acc[pr][gi][0] = 0.f; acc[pr][gi][1] = 0.f; acc[pr][gi][2] = 0.f; acc[pr][gi][3] = 0.f; }
#pragma unroll
    for (int half = 0; half < G / 2; ++half) {           // groups 2*half, 2*half+1: a 16-byte piece per token row
      uint4 kw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) kw[i] = kc4[i * 16 * G + half * 32 + g * 4 + tid];
#pragma unroll
      for (int j = 0; j < 4; ++j) {                      // word p = 4*half + j: group 2*half + j/2
        const uint4 b = qb[(4 * half + j) * 32];
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
          const uint4 &k0 = kw[2 * pr], &k1 = kw[2 * pr + 1];
          const uint32_t w0 = j == 0 ? k0.x : j == 1 ? k0.y : j == 2 ? k0.z : k0.w;
          const uint32_t w1 = j == 0 ? k1.x : j == 1 ? k1.y : j == 2 ? k1.z : k1.w;
          const uint32_t h0 = w0 >> 8, h1 = w1 >> 8;
          float (&a)[4] = acc[pr][2 * half + (j >> 1)];
          mma_f16(a, w0 & kMaskLo, w1 & kMaskLo, w0 & kMaskHi, w1 & kMaskHi, b.x, b.y);
          mma_f16(a, h0 & kMaskLo, h1 & kMaskLo, h0 & kMaskHi, h1 & kMaskHi, b.z, b.w);
        }
      }
    }
    if (G & 1) {                                         // the last group of an odd count: an 8-byte piece per token row
      uint2 kw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        kw[i] = reinterpret_cast<const uint2*>(chunk)[(i * 64 * G + (G / 2) * 128) / 2 + g * 4 + tid];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const uint4 b = qb[(4 * (G / 2) + j) * 32];
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
          const uint32_t w0 = j == 0 ? kw[2 * pr].x : kw[2 * pr].y;
          const uint32_t w1 = j == 0 ? kw[2 * pr + 1].x : kw[2 * pr + 1].y;
          const uint32_t h0 = w0 >> 8, h1 = w1 >> 8;
          float (&a)[4] = acc[pr][G - 1];
          mma_f16(a, w0 & kMaskLo, w1 & kMaskLo, w0 & kMaskHi, w1 & kMaskHi, b.x, b.y);
          mma_f16(a, h0 & kMaskLo, h1 & kMaskLo, h0 & kMaskHi, h1 & kMaskHi, b.z, b.w);
        }
      }
    }
    // the token's scale meets the integer dot products, its bias the per-group query sums
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float ks[G], kb[G];
      if (G == 3) {
        const uint32_t* v = reinterpret_cast<const uint32_t*>(ksb + (i * 8 + g) * 12);
#pragma unroll
        for (int gi = 0; gi < 3; ++gi) { const float2 f = sb_to_f2<kBf>(v[gi]); ks[gi] = f.x; kb[gi] = f.y; }
      } else if (G == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(ksb + (i * 8 + g) * 8);
        const float2 f0 = sb_to_f2<kBf>(v.x), f1 = sb_to_f2<kBf>(v.y);
        ks[0] = f0.x; kb[0] = f0.y; ks[1] = f1.x; kb[1] = f1.y;
      } else {
        const uint4 v = *reinterpret_cast<const uint4*>(ksb + (i * 8 + g) * 16);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int gi = 0; gi < 4; ++gi) { const float2 f = sb_to_f2<kBf>(u[gi]); ks[gi] = f.x; kb[gi] = f.y; }
      }
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float t = acc[i >> 1][0][2 * (i & 1) + c] * ks[0], u = qs[c][0] * kb[0];
#pragma unroll
        for (int gi = 1; gi < G; ++gi) { t = fmaf(acc[i >> 1][gi][2 * (i & 1) + c], ks[gi], t); u = fmaf(qs[c][gi], kb[gi], u); }
        sc[i][c] = fmaf(kap[c], t, u);
      }
    }
  }
  if (edge) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int pos = pos0 + 4 * g + i;
      if (pos < key_lo || pos >= key_n) { sc[i][0] = -INFINITY; sc[i][1] = -INFINITY; }
    }
  }
  // ---- online softmax over the chunk ----
  float p[4][2], corr[2];
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    float cm = fmaxf(fmaxf(sc[0][c], sc[1][c]), fmaxf(sc[2][c], sc[3][c]));
    cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 4));
    cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 8));
    cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 16));
    float m_new = fmaxf(st.m[c], cm);
    if (m_new == -INFINITY) m_new = 0.f;
    corr[c] = fast_exp2(st.m[c] - m_new);
    st.m[c] = m_new;
    p[0][c] = fast_exp2(sc[0][c] - m_new);
    p[1][c] = fast_exp2(sc[1][c] - (m_new + 4.f));       // odd token rows: p / 16 (their value codes carry a factor 16)
    p[2][c] = fast_exp2(sc[2][c] - m_new);
    p[3][c] = fast_exp2(sc[3][c] - (m_new + 4.f));
    st.l_e[c] = fmaf(st.l_e[c], corr[c], p[0][c] + p[2][c]);
    st.l_o[c] = fmaf(st.l_o[c], corr[c], p[1][c] + p[3][c]);
  }
  // rescale the accumulators when any head's running maximum moved (the lane owns the same two columns there)
  if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int gi = 0; gi < Gv; ++gi) { st.bias_e[c][gi] *= corr[c]; st.bias_o[c][gi] *= corr[c]; }
#pragma unroll
    for (int mt = 0; mt < Dv / 16; ++mt) { st.o[mt][0] *= corr[0]; st.o[mt][1] *= corr[1]; st.o[mt][2] *= corr[0]; st.o[mt][3] *= corr[1]; }
  }
  // ---- p * s_v per group as two-term binary16 (columns 0..3: high part, columns 4..7: low part), transposed into
  // the B operand of the value product: bfr[group][token row] = half2(tokens 8 tid + i, 8 tid + 4 + i) of column g ----
  uint32_t bfr[Gv][4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float vs[Gv], vb[Gv];
    if (Gv == 2) {
      const uint2 v = *reinterpret_cast<const uint2*>(vsb + (i * 8 + g) * 8);
      const float2 f0 = sb_to_f2<kBf>(v.x), f1 = sb_to_f2<kBf>(v.y);
      vs[0] = f0.x; vb[0] = f0.y; vs[1] = f1.x; vb[1] = f1.y;
    } else {
      const uint4 v = *reinterpret_cast<const uint4*>(vsb + (i * 8 + g) * 16);
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int gi = 0; gi < 4; ++gi) { const float2 f = sb_to_f2<kBf>(u[gi]); vs[gi] = f.x; vb[gi] = f.y; }
    }
    if (edge) {
      const int pos = pos0 + 4 * g + i;
      if (pos < key_lo || pos >= key_n) {
#pragma unroll
        for (int gi = 0; gi < Gv; ++gi) { vs[gi] = 0.f; vb[gi] = 0.f; }
      }
    }
#pragma unroll
    for (int gi = 0; gi < Gv; ++gi) {
      const float x0 = p[i][0] * vs[gi], x1 = p[i][1] * vs[gi];
      // columns 0..3: trunc16(x); columns 4..7: trunc16(x - trunc11bits(x)) -- the binary16 conversion truncates
      const float r0 = x0 - __uint_as_float(__float_as_uint(x0) & split_mask);
      const float r1 = x1 - __uint_as_float(__float_as_uint(x1) & split_mask);
      bfr[gi][i] = transpose_8x8_b16(f32x2_to_h2_rz(r0, r1));
      if (i & 1) {
        st.bias_o[0][gi] = fmaf(p[i][0], vb[gi], st.bias_o[0][gi]);
        st.bias_o[1][gi] = fmaf(p[i][1], vb[gi], st.bias_o[1][gi]);
      } else {
        st.bias_e[0][gi] = fmaf(p[i][0], vb[gi], st.bias_e[0][gi]);
        st.bias_e[1][gi] = fmaf(p[i][1], vb[gi], st.bias_e[1][gi]);
      }
    }
  }
  // ---- P.V on the codes: 16 value rows x 8 columns (heads hi|lo) x 32 tokens per tile pair ----
#pragma unroll
  for (int q4 = 0; q4 < Dv / 32; ++q4) {
    const uint4 w4 = vc4[(q4 * 8 + g) * 4 + tid];
    const int gi = q4 >> 1;
    {
      const uint32_t xh = w4.x >> 8, yh = w4.y >> 8;
      mma_f16(st.o[2 * q4], w4.x & kMaskLo, w4.y & kMaskLo, w4.x & kMaskHi, w4.y & kMaskHi, bfr[gi][0], bfr[gi][1]);
      mma_f16(st.o[2 * q4], xh & kMaskLo, yh & kMaskLo, xh & kMaskHi, yh & kMaskHi, bfr[gi][2], bfr[gi][3]);
    }
    {
      const uint32_t xh = w4.z >> 8, yh = w4.w >> 8;
      mma_f16(st.o[2 * q4 + 1], w4.z & kMaskLo, w4.w & kMaskLo, w4.z & kMaskHi, w4.w & kMaskHi, bfr[gi][0], bfr[gi][1]);
      mma_f16(st.o[2 * q4 + 1], xh & kMaskLo, yh & kMaskLo, xh & kMaskHi, yh & kMaskHi, bfr[gi][2], bfr[gi][3]);
    }
  }
}

__device__ inline void store_out(const DecodeParams& P, size_t index, float v) {
  if (P.out_dtype == Q4KV_OUT_BF16) reinterpret_cast<__nv_bfloat16*>(P.out)[index] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(P.out)[index] = v;
}

// Epilogue of one segment, run by the single warp that made the deposit count complete: combine
// the NW deposits; a pair that lies wholly inside this CTA is normalised and written out, otherwise
// the combination becomes this CTA's partial record and the warp takes a ticket -- the CTA whose
// ticket is the pair's last combines all records of the pair.  Each lane owns 4 consecutive output
// elements (per 128), so every access is a 16-byte one.  Deposits and records are walked in loops with a
// few loads in flight and running sums in registers: the register need does not grow with the number of
// warps or records.
template <int G, int NW>
__device__ __forceinline__ void segment_epilogue(const float* merge_buf, int* epilogues_word, int use, const DecodeParams& P,
                                              const Segment& seg, int cta, const Partition& part, int lane) {
  constexpr int Dv = 64 * value_groups(G), V = Dv / 128;
  constexpr int kStride = Dv + 8;
  static_assert(NW <= 32, "one lane per deposit in the weight pass");
  const Layout& y = P.y;
  const int n_rep = y.n_rep;
  const int pair = seg.a * y.Hkv + seg.hk;
  const bool whole = seg.c0 == seg.cf && seg.c1 == seg.cf + seg.nc;
  const size_t row0 = (size_t)seg.a * y.Hq + (size_t)seg.hk * n_rep;
  const size_t rstride = (size_t)n_rep * kRecStride(Dv);
  float* rec = P.partials + (size_t)(pair + cta) * rstride;
  auto store4 = [&](int h, int d, float4 v) {
    if (P.out_dtype == Q4KV_OUT_BF16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      uint2 u = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(P.out) + (row0 + h) * Dv + d) = u;
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(P.out) + (row0 + h) * Dv + d) = v;
    }
  };
  // weights of the deposits, all heads side by side: lane w looks at deposit w
  float wgt[4], Mh[4], Lh[4];
  bool badh[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    const float* mine = merge_buf + ((size_t)(lane < NW ? lane : 0) * 4 + h) * kStride;
    const float2 ml = *reinterpret_cast<const float2*>(mine + Dv);
    const float mw = (lane < NW && h < n_rep) ? ml.x : -INFINITY, lw = (lane < NW && h < n_rep) ? ml.y : 0.f;
    float M = mw;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    wgt[h] = mw == -INFINITY ? 0.f : fast_exp2(mw - M);
    float L = wgt[h] * lw;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
    badh[h] = __any_sync(0xffffffffu, lw < 0.f);
    Mh[h] = M;
    Lh[h] = badh[h] ? 0.f : L;
  }
  float4 acc[4][V];
#pragma unroll
  for (int h = 0; h < 4; ++h)
#pragma unroll
    for (int v = 0; v < V; ++v) acc[h][v] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
  for (int w = 0; w < NW; ++w) {
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const float ww = __shfl_sync(0xffffffffu, wgt[h], w);
      const bool on = ww != 0.f;                         // an empty deposit holds stale bytes
      const float* dep = merge_buf + ((size_t)w * 4 + h) * kStride;
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const float4 x = *reinterpret_cast<const float4*>(dep + 128 * v + 4 * lane);
        const float bs = dep[Dv + 2 + ((128 * v + 4 * lane) >> 6)];
        acc[h][v].x = fmaf(ww, on ? x.x + bs : 0.f, acc[h][v].x); acc[h][v].y = fmaf(ww, on ? x.y + bs : 0.f, acc[h][v].y);
        acc[h][v].z = fmaf(ww, on ? x.z + bs : 0.f, acc[h][v].z); acc[h][v].w = fmaf(ww, on ? x.w + bs : 0.f, acc[h][v].w);
      }
    }
  }
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    if (h >= n_rep) continue;
    const float inv = whole ? (Lh[h] > 0.f ? 1.f / Lh[h] : 0.f) : 1.f;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      float4 o = acc[h][v];
      o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
      const int d = 128 * v + 4 * lane;
      if (whole) store4(h, d, o);
      else *reinterpret_cast<float4*>(rec + (size_t)h * kRecStride(Dv) + d) = o;
    }
    if (lane == 0) {
      if (whole) { if (P.lse) P.lse[row0 + h] = Lh[h] > 0.f ? (Mh[h] + log2f(Lh[h])) / kLog2e : -INFINITY; }
      else *reinterpret_cast<float2*>(rec + (size_t)h * kRecStride(Dv) + Dv) = make_float2(Mh[h], badh[h] ? -1.f : Lh[h]);
    }
  }
  // the deposit buffer can be reused from here on
  __threadfence_block();
  __syncwarp();
  if (lane == 0) *(volatile int*)epilogues_word = use + 1;
  if (whole) return;

  // ticket: the CTA whose record arrives last combines all records of the pair
  const uint32_t pair_u0 = seg.u0 - (uint32_t)(seg.c0 - seg.cf);
  const int c_first = part.cta_of(pair_u0), c_last = part.cta_of(pair_u0 + (uint32_t)seg.nc - 1u);
  // The warp's record stores are ordered before lane 0's release by the warp barrier, and the other lanes' record loads
  // after its acquire by the second one: one acquire-release atomic takes the place of a fence on either side.
  __syncwarp();
  int final_merge = 0;
  if (lane == 0) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(&P.tickets[pair]) : "memory");
    final_merge = old == c_last - c_first;
    if (final_merge) P.tickets[pair] = 0;            // ready for the next call
  }
  final_merge = __shfl_sync(0xffffffffu, final_merge, 0);
  if (!final_merge) return;
  __syncwarp();
  const int R = c_last - c_first + 1;
  const float* base = P.partials + (size_t)(pair + c_first) * rstride;
  // The records sit in L2, a microsecond away: all heads travel together, and the first batch of record loads is issued
  // before the (m, l) pass, so that a pair with few records costs two round trips in all.
  constexpr int RB = V == 1 ? 5 : 2;
  float mr[RB][4];
  float4 xv[RB][4][V];
  auto load_batch = [&](int rb) {
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      const int r = rb + i < R ? rb + i : R - 1;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const float* rh = base + r * rstride + (size_t)(h < n_rep ? h : 0) * kRecStride(Dv);
        mr[i][h] = __ldcg(rh + Dv);
#pragma unroll
        for (int v = 0; v < V; ++v) xv[i][h][v] = __ldcg(reinterpret_cast<const float4*>(rh + 128 * v + 4 * lane));
      }
    }
  };
  load_batch(0);
  // pass 1: maximum and sum per head.  Lane l looks at (record, head) pairs l, l + 32, ...; its head is l % 4.
  const int hl = lane & 3;
  float Ml = -INFINITY, Ll = 0.f;
  int badl = 0;
  if (hl < n_rep) {
    for (int r = lane >> 2; r < R; r += 8) {
      const float2 t = __ldcg(reinterpret_cast<const float2*>(base + r * rstride + (size_t)hl * kRecStride(Dv) + Dv));
      if (t.y < 0.f) badl = 1;
      const float Mn = fmaxf(Ml, t.x);
      if (Mn != -INFINITY) Ll = Ll * fast_exp2(Ml - Mn) + t.y * fast_exp2(t.x - Mn);
      Ml = Mn;
    }
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    const float Mo = __shfl_xor_sync(0xffffffffu, Ml, o), Lo = __shfl_xor_sync(0xffffffffu, Ll, o);
    const float Mn = fmaxf(Ml, Mo);
    if (Mn != -INFINITY) Ll = Ll * fast_exp2(Ml - Mn) + Lo * fast_exp2(Mo - Mn);
    Ml = Mn;
  }
  const bool any_bad = __any_sync(0xffffffffu, badl);
  // pass 2: weighted sum of the records, RB at a time, all heads together (nothing is stored before the end)
  float Mr[4], Lr[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    Mr[h] = __shfl_sync(0xffffffffu, Ml, h);
    Lr[h] = any_bad ? 0.f : __shfl_sync(0xffffffffu, Ll, h);
  }
  float4 racc[4][V];
#pragma unroll
  for (int h = 0; h < 4; ++h)
#pragma unroll
    for (int v = 0; v < V; ++v) racc[h][v] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int rb = 0; rb < R; rb += RB) {
    if (rb > 0) load_batch(rb);
#pragma unroll
    for (int i = 0; i < RB; ++i)
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const float e = (rb + i >= R || mr[i][h] == -INFINITY) ? 0.f : fast_exp2(mr[i][h] - Mr[h]);
#pragma unroll
        for (int v = 0; v < V; ++v) {
          racc[h][v].x = fmaf(e, xv[i][h][v].x, racc[h][v].x); racc[h][v].y = fmaf(e, xv[i][h][v].y, racc[h][v].y);
          racc[h][v].z = fmaf(e, xv[i][h][v].z, racc[h][v].z); racc[h][v].w = fmaf(e, xv[i][h][v].w, racc[h][v].w);
        }
      }
  }
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    if (h >= n_rep) continue;
    const float inv = Lr[h] > 0.f ? 1.f / Lr[h] : 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      float4 o = racc[h][v];
      o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
      store4(h, 128 * v + 4 * lane, o);
    }
    if (lane == 0 && P.lse) P.lse[row0 + h] = Lr[h] > 0.f ? (Mr[h] + log2f(Lr[h])) / kLog2e : -INFINITY;
  }
}

// Epilogue of a CTA's last segment, one warp per query head (warp h < n_rep handles head h; the caller has waited for
// all NW deposits).  Same arithmetic as segment_epilogue; the heads run side by side instead of one after the other,
// which shortens the tail every launch ends with: combine, record, ticket, final combination.  The head warps meet
// twice through shared memory: once so that a single thread draws the pair's ticket after all heads' records are
// written and fenced, once to learn whether this CTA combines the pair's records.
template <int G, int NW>
__device__ __forceinline__ void last_segment_by_heads(const float* merge_buf, int* fin_arrived, int* fin_ticket,
                                                      volatile int* abort_flag, const DecodeParams& P, const Segment& seg,
                                                      int cta, const Partition& part, int h, int lane) {
  constexpr int Dv = 64 * value_groups(G), V = Dv / 128;
  constexpr int kStride = Dv + 8;
  const Layout& y = P.y;
  const int n_rep = y.n_rep;
  const int pair = seg.a * y.Hkv + seg.hk;
  const bool whole = seg.c0 == seg.cf && seg.c1 == seg.cf + seg.nc;
  const size_t row = (size_t)seg.a * y.Hq + (size_t)seg.hk * n_rep + h;
  const size_t rstride = (size_t)n_rep * kRecStride(Dv);
  float* rec = P.partials + (size_t)(pair + cta) * rstride + (size_t)h * kRecStride(Dv);
  auto store4 = [&](int d, float4 v) {
    if (P.out_dtype == Q4KV_OUT_BF16) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      uint2 u = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(P.out) + row * Dv + d) = u;
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(P.out) + row * Dv + d) = v;
    }
  };
  // weights of the deposits: lane w looks at deposit w
  const float* mine = merge_buf + ((size_t)(lane < NW ? lane : 0) * 4 + h) * kStride;
  const float2 ml = *reinterpret_cast<const float2*>(mine + Dv);
  const float mw = lane < NW ? ml.x : -INFINITY, lw = lane < NW ? ml.y : 0.f;
  float M = mw;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  const float wgt = mw == -INFINITY ? 0.f : fast_exp2(mw - M);
  float L = wgt * lw;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  const bool bad = __any_sync(0xffffffffu, lw < 0.f);
  if (bad) L = 0.f;
  float4 acc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int w = 0; w < NW; ++w) {
    const float ww = __shfl_sync(0xffffffffu, wgt, w);
    const bool on = ww != 0.f;                           // an empty deposit holds stale bytes
    const float* dep = merge_buf + ((size_t)w * 4 + h) * kStride;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const float4 x = *reinterpret_cast<const float4*>(dep + 128 * v + 4 * lane);
      const float bs = dep[Dv + 2 + ((128 * v + 4 * lane) >> 6)];
      acc[v].x = fmaf(ww, on ? x.x + bs : 0.f, acc[v].x); acc[v].y = fmaf(ww, on ? x.y + bs : 0.f, acc[v].y);
      acc[v].z = fmaf(ww, on ? x.z + bs : 0.f, acc[v].z); acc[v].w = fmaf(ww, on ? x.w + bs : 0.f, acc[v].w);
    }
  }
  if (whole) {
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) store4(128 * v + 4 * lane, make_float4(acc[v].x * inv, acc[v].y * inv, acc[v].z * inv, acc[v].w * inv));
    if (lane == 0 && P.lse) P.lse[row] = L > 0.f ? (M + log2f(L)) / kLog2e : -INFINITY;
    return;
  }
#pragma unroll
  for (int v = 0; v < V; ++v) *reinterpret_cast<float4*>(rec + 128 * v + 4 * lane) = acc[v];
  if (lane == 0) *reinterpret_cast<float2*>(rec + Dv) = make_float2(M, bad ? -1.f : L);
  // every head's record is written and fenced before one thread draws the ticket
  const uint32_t pair_u0 = seg.u0 - (uint32_t)(seg.c0 - seg.cf);
  const int c_first = part.cta_of(pair_u0), c_last = part.cta_of(pair_u0 + (uint32_t)seg.nc - 1u);
  // Ordering: each head warp's record stores come before its lane 0's arrival (warp barrier, then a CTA-scope
  // fence); the last arrival draws the ticket with one acquire-release atomic at GPU scope, which publishes all the
  // head warps' records and, if the ticket is the pair's last, makes the other CTAs' records readable; the answer
  // reaches the other head warps through shared memory and a CTA-scope fence.
  __syncwarp();
  int state = 0;
  if (lane == 0) {
    __threadfence_block();
    if (atomicAdd(fin_arrived, 1) == n_rep - 1) {
      __threadfence_block();
      int old;
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(&P.tickets[pair]) : "memory");
      const int final_merge = old == c_last - c_first;
      if (final_merge) P.tickets[pair] = 0;          // ready for the next call
      __threadfence_block();
      *(volatile int*)fin_ticket = 1 + final_merge;
    }
    for (uint32_t i = 0; i < (kSpinLimit << 4) && (state = *(volatile int*)fin_ticket) == 0; ++i)
      if ((i & 255u) == 255u && *abort_flag) break;
    __threadfence_block();
  }
  state = __shfl_sync(0xffffffffu, state, 0);
  if (state != 2) return;
  __syncwarp();
  // this CTA drew the pair's last ticket: head h of all records, the loads of up to RB records in flight together
  const int R = c_last - c_first + 1;
  const float* base = P.partials + (size_t)(pair + c_first) * rstride + (size_t)h * kRecStride(Dv);
  constexpr int RB = V == 1 ? 8 : 4;
  float Mr = -INFINITY, Lr = 0.f;
  bool any_bad = false;
  float4 racc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) racc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int rb = 0; rb < R; rb += RB) {
    float2 mlr[RB];
    float4 xv[RB][V];
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      const float* rh = base + (size_t)(rb + i < R ? rb + i : R - 1) * rstride;
      mlr[i] = __ldcg(reinterpret_cast<const float2*>(rh + Dv));
#pragma unroll
      for (int v = 0; v < V; ++v) xv[i][v] = __ldcg(reinterpret_cast<const float4*>(rh + 128 * v + 4 * lane));
    }
    float Mn = Mr;
#pragma unroll
    for (int i = 0; i < RB; ++i) if (rb + i < R) Mn = fmaxf(Mn, mlr[i].x);
    const float c0 = Mn == -INFINITY ? 0.f : fast_exp2(Mr - Mn);      // Mr = -inf gives 0
    Lr *= c0;
#pragma unroll
    for (int v = 0; v < V; ++v) { racc[v].x *= c0; racc[v].y *= c0; racc[v].z *= c0; racc[v].w *= c0; }
#pragma unroll
    for (int i = 0; i < RB; ++i) {
      if (rb + i >= R) continue;
      if (mlr[i].y < 0.f) any_bad = true;
      const float e = mlr[i].x == -INFINITY ? 0.f : fast_exp2(mlr[i].x - Mn);
      Lr = fmaf(e, mlr[i].y, Lr);
#pragma unroll
      for (int v = 0; v < V; ++v) {
        racc[v].x = fmaf(e, xv[i][v].x, racc[v].x); racc[v].y = fmaf(e, xv[i][v].y, racc[v].y);
        racc[v].z = fmaf(e, xv[i][v].z, racc[v].z); racc[v].w = fmaf(e, xv[i][v].w, racc[v].w);
      }
    }
    Mr = Mn;
  }
  if (any_bad) Lr = 0.f;
  const float inv = Lr > 0.f ? 1.f / Lr : 0.f;
#pragma unroll
  for (int v = 0; v < V; ++v) store4(128 * v + 4 * lane, make_float4(racc[v].x * inv, racc[v].y * inv, racc[v].z * inv, racc[v].w * inv));
  if (lane == 0 && P.lse) P.lse[row] = Lr > 0.f ? (Mr + log2f(Lr)) / kLog2e : -INFINITY;
}

template <int G, int NW, bool kBf>
__global__ void __launch_bounds__((NW + 1) * 32, 1) decode_mma_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int Gv = value_groups(G), Dv = 64 * Gv;
  using S = Smem<G, NW>;
  constexpr int kSlots = S::kSlots, kChunkBytes = S::kChunkBytes, kMBufs = S::kMBufs;
  static_assert(kSlots >= NW + 4, "the ring must hold the chunks in work and a few in flight");
  extern __shared__ __align__(128) uint8_t smem_raw[];
  S& sm = *reinterpret_cast<S*>(smem_raw);

  const Layout& y = P.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const int n_rep = y.n_rep;

  grid_launch_dependents();
  // rows of query heads that do not exist (n_rep < 4) are never staged: they stay zero
  for (int i = threadIdx.x; i < kQBufs * 2 * G * 32; i += blockDim.x) (&sm.qfrag[0][0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.full[s], 1); sm.released[s] = 0; sm.bad[s] = 0; sm.patched[s] = 0; }
    for (int i = 0; i < kQBufs; ++i) sm.q_tag[i] = 0;
    for (int i = 0; i < kMBufs; ++i) { sm.deposits[i] = 0; sm.epilogues[i] = 0; sm.epi_claim[i] = 0; }
    sm.all_issued = 0;
    sm.next_chunk = 0;
    sm.fin_arrived = 0; sm.fin_ticket = 0;
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  // ---- this CTA's unit range (every warp computes it for itself; these inputs are not written by any kernel) ----
  const RangeStart rs = find_range(P, cta, gridDim.x);
  if (rs.any_bad && cta == 0 && threadIdx.x == 0) raise_flag(P.flags, Q4KV_FLAG_BAD_LENGTH);
  const int n_chunks = (int)(rs.u_end - rs.u_begin);
  Walker wk;
  wk.init(P, rs);
  Segment seg;

  const uint8_t* layer_base = P.pool + (uint64_t)P.layer * y.layer_bytes;
  // hand ring slot `slot` to the chunk whose table entry is `off`
  auto issue_copy = [&](int slot, uint32_t off) {
    if (off == kOffBad) {
      sm.bad[slot] = 1;
      mbar_arrive(&sm.full[slot]);
    } else {
      sm.bad[slot] = 0;
      mbar_arrive_expect_tx(&sm.full[slot], kChunkBytes);
      bulk_load(sm.ring + (size_t)slot * kChunkBytes, layer_base + (uint64_t)off * 16u, kChunkBytes, &sm.full[slot]);
    }
  };

  // =============================== planner warp ================================================
  if (warp == NW) {
    // Planning step: 32 chunks, one per lane: block-table entry -> pool offset -> table entry k % kOffCap.  Issue
    // step: lane s owns ring slot s and the chunks s, s + kSlots, ...; it copies its next chunk once the slot's
    // previous chunk has been consumed and the chunk has its table entry.  All lanes follow one path.  Lengths and
    // block tables are inputs that no kernel writes, so the first planning steps run while the preceding kernel drains;
    // the pool is read only after it.
    static_assert(kSlots <= 32 && kOffCap >= 2 * 32 + kSlots, "table ring: a step of entries ahead of every reader");
    // Once every chunk has been issued this warp has time to spare, and it takes the epilogues of the segments that
    // complete from then on (all but the CTA's last): a consumer that leaves the stream for an epilogue (a few
    // microseconds with the ticket and a pair's final combination) costs its CTA an extra round of chunks.  While
    // chunks are still to be issued the consumers keep them, or the ring would run dry meanwhile.  A claim word per
    // deposit buffer decides who runs one.  Segments complete in order, so a second walker names the next one.
    // d = 128 only (5 agents x 4097 tokens: 20.2 -> 19.2 us per launch, 2 agents: 18.4 -> 15.9 us; 40 agents: 1.8 %
    // slower): in the other instantiations the second copy of the epilogue's code slowed the chunk loop of long
    // launches by 5-9 %, as one shared non-inlined copy did through its spills.
    // (A segment is the CTA's last when its chunks end the CTA's range: no count of the segments is needed.)
    Walker wke = wk;
    Segment sge;
    int epi_idx = 0;
    bool epi_more = false, epi_started = false;          // sge names a segment that is not the CTA's last
    bool waited = false, bad_block = false, more = wk.next(seg), all_out = false;
    int tq_head = 0, tq_tail = 0;            // patch queue: entries tq_head .. tq_tail-1 (indices taken modulo kTailQ)
    int kb = 0;                              // chunks of `seg` already planned
    int planned = 0;                         // chunks of the CTA that have their table entry
    int next_k = lane < kSlots ? lane : INT_MAX, round = 0;   // this lane's next chunk and its round in the slot
    const volatile int* my_released = &sm.released[lane < kSlots ? lane : 0];
    uint32_t idle = 0;
    for (;;) {
      // ---- plan as far as the table allows: entries below every lane's next chunk are dead ----
      if (more) {
        int lo = next_k;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        while (more && planned + 32 <= lo + kOffCap && tq_tail - tq_head < kTailQ) {
          const int cnt = seg.c1 - seg.c0;
          if (kb == 0 && seg.tail_pos >= 0) {
            // this segment ends with the agent's newest position: queue the patch, ask for the new rows
            if (lane == 0) sm.tail_q[tq_tail % kTailQ] = make_int4(seg.k0 + seg.tail_pos, seg.a, seg.hk, (seg.n - 1) & 31);
            ++tq_tail;
            prefetch_new_token<G>(P.k_new, P.v_new, y.Hkv, seg.a, seg.hk, lane);
          }
          if (kb + lane < cnt) {
            const int c = seg.chunk_at(kb + lane);
            const int blk = P.tables[(size_t)seg.ar * P.max_blocks + (c >> 3)];
            uint32_t off = kOffBad;
            if (blk >= 0 && blk < P.n_blocks)
              off = (uint32_t)(((uint64_t)seg.li * y.layer_bytes + (uint64_t)blk * y.block_bytes + (uint64_t)seg.hk * y.head_block_bytes +
                                (uint64_t)(c & 7) * kChunkBytes) >> 4);
            else
              bad_block = true;
            sm.src_off[(seg.k0 + kb + lane) % kOffCap] = off;
          }
          kb += 32;
          if (kb >= cnt) { planned = seg.k0 + cnt; kb = 0; more = wk.next(seg); } else { planned = seg.k0 + kb; }
        }
        __syncwarp();
      }
      if (!waited) {
        // While the preceding kernel drains, ask L2 for the chunks of the first ring fill (more than that was measured
        // and is no faster; the same prefetch in the MLA-latent kernel gains nothing).  A prefetch returns nothing
        // to the kernel, and L2 is where the preceding kernel's writes land, so what the copies read after the wait
        // is current whatever that kernel still writes.
        if (lane < kSlots && next_k < planned) {
          const uint32_t off = sm.src_off[next_k % kOffCap];
          if (off != kOffBad) prefetch_l2_bulk(layer_base + (uint64_t)off * 16u, kChunkBytes);
        }
        grid_dependency_wait();
        waited = true;
      }
      // ---- issue: a short polling loop, left from time to time to plan further ----
      bool any_left = true;
      for (int it = 0; it < 64 && any_left; ++it) {
        // the fused append: quantize the new token into the oldest queued chunk once that chunk has landed (the whole
        // warp works on it; its consumer waits for sm.patched)
        if (tq_head < tq_tail) {
          const int4 t = sm.tail_q[tq_head % kTailQ];
          const int tslot = t.x % kSlots, tround = t.x / kSlots;
          const int issued = __shfl_sync(0xffffffffu, round, tslot);      // copies this slot's lane has issued so far
          if (issued > tround && mbar_test_wait(&sm.full[tslot], (uint32_t)tround & 1u)) {
            if (!sm.bad[tslot]) {
              uint8_t* gchunk = const_cast<uint8_t*>(layer_base) + (uint64_t)sm.src_off[t.x % kOffCap] * 16u;
              append_new_token<G>(sm.ring + (size_t)tslot * kChunkBytes, gchunk, y, P.k_new, P.v_new, t.y, t.z, t.w, lane);
            }
            __threadfence_block();
            __syncwarp();
            if (lane == 0) *(volatile int*)&sm.patched[tslot] = tround + 1;
            ++tq_head;
            idle = 0;
          }
        }
        if (G == 2 && epi_more) {
          const int eb = epi_idx % kMBufs, euse = epi_idx / kMBufs;
          if (*(volatile int*)&sm.deposits[eb] >= (euse + 1) * NW) {
            int state = 0;                               // 1: a consumer has it, 2: this warp takes it
            if (lane == 0) {
              if (*(volatile int*)&sm.epi_claim[eb] > euse) state = 1;
              else if (all_out) state = atomicCAS(&sm.epi_claim[eb], euse, euse + 1) == euse ? 2 : 1;
            }
            state = __shfl_sync(0xffffffffu, state, 0);
            if (state == 2) {
              __threadfence_block();
              segment_epilogue<G, NW>(&sm.merge[eb][0][0][0], &sm.epilogues[eb], euse, P, sge, cta, rs.part, lane);
            }
            if (state != 0) {
              epi_more = wke.next(sge) && sge.k0 + (sge.c1 - sge.c0) < n_chunks;
              ++epi_idx;
              idle = 0;
            }
          }
        }
        const bool can = next_k < planned && *my_released >= round;
        if (can) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the consumer's reads and patches of the slot come first
          issue_copy(lane, sm.src_off[next_k % kOffCap]);
          next_k += kSlots;
          ++round;
        }
        if (G == 2 && !epi_started) {                    // the first segment is named here, after the first copies are out
          epi_started = true;
          epi_more = wke.next(sge) && sge.k0 + (sge.c1 - sge.c0) < n_chunks;
        }
        if (!all_out && !__any_sync(0xffffffffu, next_k < n_chunks)) {
          all_out = true;
          if (lane == 0) *(volatile int*)&sm.all_issued = 1;
        }
        any_left = !all_out || tq_head < tq_tail || (G == 2 && epi_more);
        if (__any_sync(0xffffffffu, can)) { idle = 0; continue; }
        if (more && tq_tail - tq_head < kTailQ && __all_sync(0xffffffffu, next_k >= planned)) break;   // plan further first
        ++idle;
        __nanosleep(200);
      }
      if (!any_left) break;                  // every chunk has been issued, every epilogue but the last is done
      if (idle > (kSpinLimit >> 2) || *(volatile int*)&sm.abort_flag) {
        if (lane == 0) { sm.abort_flag = 1; raise_flag(P.flags, Q4KV_FLAG_INTERNAL); }
        // giving up: each lane lets the last copy it issued into its slot land before the CTA lets go of shared memory
        if (lane < kSlots && round > 0)
          for (uint32_t i = 0; i < 4096u && !mbar_try_wait(&sm.full[lane], (uint32_t)(round - 1) & 1u); ++i) {}
        break;
      }
    }
    if (bad_block) raise_flag(P.flags, Q4KV_FLAG_BAD_BLOCK);
    return;
  }

  // =============================== consumer warps ==============================================
  // Everything the consumers write (output rows, partial records, tickets) may still be in use by
  // the preceding kernels of the stream until they have completed.
  grid_dependency_wait();
  const int g = lane >> 2, tid = lane & 3;
  // this lane's two score columns 2 tid, 2 tid + 1 of eight: columns 0..3 are the query heads of the KV head, 4..7
  // repeat them and carry p*s minus its binary16 truncation
  const int hcol[2] = {(2 * tid) & 3, (2 * tid + 1) & 3};
  const bool live[2] = {hcol[0] < n_rep, hcol[1] < n_rep};
  const uint32_t split_mask = tid >= 2 ? 0xFFFFE000u : 0u;

  // agents without any key (kv_len == 0 or a rejected length): zeros, lse = -inf
  for (int a = cta * NW + warp; a < P.n_agents; a += gridDim.x * NW) {
    bool bad_len;
    if (agent_range(P, a, bad_len).nc > 0) continue;
    for (int i = lane; i < y.Hq * Dv; i += 32) store_out(P, (size_t)a * y.Hq * Dv + i, 0.f);
    if (P.lse) for (int i = lane; i < y.Hq; i += 32) P.lse[(size_t)a * y.Hq + i] = -INFINITY;
  }
  if (n_chunks == 0) return;

  // ---- the first segments' queries are staged up front, one warp each ----
  {
    Walker w2 = wk;
    Segment s2;
    for (int s = 0; s < kQBufs && w2.next(s2); ++s) {
      if (s % NW != warp) continue;
      stage_query<G>(sm.qfrag[s], sm.qsum[s], sm.kappa[s], P.q, y.Hq, n_rep, P.scale_log2, s2.a, s2.hk, lane);
      __threadfence_block();
      __syncwarp();
      if (lane == 0) *(volatile int*)&sm.q_tag[s] = s + 1;
    }
  }

  bool aborted = false, poisoned = false;
  int cur = -1;                 // index of the segment `seg` describes (-1: none yet)
  bool have_seg = false;        // this warp holds state for segment `cur`
  const uint4* qa = nullptr;    // this lane's A registers of the segment's query, in shared memory
  float qs[2][G], kap[2] = {0.f, 0.f};
  WarpState<G> st;
  st.reset();

  // Deposit this warp's state for segment `cur` (described by `seg`); the warp that completes the
  // count combines the deposits and runs the segment's epilogue.
  auto deposit_and_maybe_finish = [&](bool real) {
    const int b = cur % kMBufs, use = cur / kMBufs;
    // the buffer is free once the epilogue of its previous use is done
    if (!aborted && !spin_until_ge(&sm.epilogues[b], use, &sm.abort_flag)) aborted = true;
    float (*mg)[S::kMergeStride] = sm.merge[b][warp];
    if (real) {
      // sums over the lane's tokens -> sums over the chunk's tokens (the eight lanes of equal tid)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float l = st.l_e[c] + 16.f * st.l_o[c];
        l += __shfl_xor_sync(0xffffffffu, l, 4);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        float bias[Gv];
#pragma unroll
        for (int gi = 0; gi < Gv; ++gi) {
          float bb = st.bias_e[c][gi] + 16.f * st.bias_o[c][gi];
          bb += __shfl_xor_sync(0xffffffffu, bb, 4);
          bb += __shfl_xor_sync(0xffffffffu, bb, 8);
          bb += __shfl_xor_sync(0xffffffffu, bb, 16);
          bias[gi] = bb;
        }
        if (g == 0 && tid < 2) {
          float* row = mg[2 * tid + c];
          row[Dv] = st.m[c];
          row[Dv + 1] = (poisoned || aborted) ? -1.f : l;
#pragma unroll
          for (int gi = 0; gi < Gv; ++gi) row[Dv + 2 + gi] = bias[gi];
        }
      }
      // columns 4..7 (lanes tid 2,3) hold the low-part products of heads 0..3
#pragma unroll
      for (int mt = 0; mt < Dv / 16; ++mt) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float v = st.o[mt][r] + __shfl_xor_sync(0xffffffffu, st.o[mt][r], 2);
          if (tid < 2) mg[2 * tid + (r & 1)][16 * mt + g + 8 * (r >> 1)] = v * 16777216.f;
        }
      }
    } else if (lane < 4) {
      mg[lane][Dv] = -INFINITY;
      mg[lane][Dv + 1] = aborted ? -1.f : 0.f;
    }
    __threadfence_block();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = atomicAdd(&sm.deposits[b], 1) == (use + 1) * NW - 1;
    last = __shfl_sync(0xffffffffu, last, 0);
    const bool last_seg = seg.k0 + (seg.c1 - seg.c0) >= n_chunks;     // this segment's chunks end the CTA's range
    if (G != 3 && last_seg) {
      // the CTA's last segment: nothing is left to stream, so the head warps wait for the last deposit and share the
      // epilogue; the other warps are done.  (Not in the d_qk 192 instantiation, where it measured 0.4 % slower.  On the
      // d-128 kernel it cost 1.2 us while a consumer still ran the epilogues of earlier segments; since the planner
      // warp takes those it saves 0.5 us per launch at 5 agents and 0.8 us at 2.)
      if (warp >= n_rep) return;
      {
        bool ok = false;
        for (uint32_t i = 0; i < (kSpinLimit << 2); ++i) {
          if (*(volatile int*)&sm.deposits[b] >= (use + 1) * NW) { ok = true; break; }
          __nanosleep(100);
          if ((i & 63u) == 63u && *(volatile int*)&sm.abort_flag) break;
        }
        if (!ok) return;
      }
      __threadfence_block();
      last_segment_by_heads<G, NW>(&sm.merge[b][0][0][0], &sm.fin_arrived, &sm.fin_ticket, &sm.abort_flag, P, seg, cta,
                                   rs.part, warp, lane);
      return;
    }
    if (!last) return;
    if (G == 2 && !last_seg) {
      // an earlier segment: the planner warp takes it if it has nothing left to issue
      int mine = 0;
      if (lane == 0 && !*(volatile int*)&sm.all_issued) mine = atomicCAS(&sm.epi_claim[b], use, use + 1) == use;
      if (!__shfl_sync(0xffffffffu, mine, 0)) return;
    }
    __threadfence_block();
    segment_epilogue<G, NW>(&sm.merge[b][0][0][0], &sm.epilogues[b], use, P, seg, cta, rs.part, lane);
  };

  // A chunk is claimed only when the warp is free to work on it: a warp that is away in a segment's epilogue (a few
  // microseconds when it merges a pair's records) must not sit on a claimed chunk meanwhile.
  bool out_of_chunks = false;
  for (;;) {
    int k = 0;
    if (!out_of_chunks) {
      if (lane == 0) k = atomicAdd(&sm.next_chunk, 1);
      k = __shfl_sync(0xffffffffu, k, 0);
      out_of_chunks = k >= n_chunks;
    }
    // move to the segment that holds chunk k (to the end of the list when out of chunks), leaving a
    // deposit in every segment passed
    bool finished = false;
    while (cur < 0 || out_of_chunks || k >= seg.k0 + (seg.c1 - seg.c0)) {
      if (cur >= 0) deposit_and_maybe_finish(have_seg);
      have_seg = false;
      poisoned = false;
      if (!wk.next(seg)) { finished = true; break; }
      ++cur;
    }
    if (finished) break;
    if (!have_seg) {
      // entering segment `cur`: its query fragments
      const int qb = cur % kQBufs;
      if (cur >= kQBufs && k == seg.k0) {
        // later segments are staged by whoever claims their first chunk, once the buffer's previous
        // segment has been left by every warp (its epilogue is done)
        const int prev = cur - kQBufs;
        if (!aborted && !spin_until_ge(&sm.epilogues[prev % kMBufs], prev / kMBufs + 1, &sm.abort_flag)) aborted = true;
        stage_query<G>(sm.qfrag[qb], sm.qsum[qb], sm.kappa[qb], P.q, y.Hq, n_rep, P.scale_log2, seg.a, seg.hk, lane);
        __threadfence_block();
        __syncwarp();
        if (lane == 0) *(volatile int*)&sm.q_tag[qb] = cur + 1;
      }
      if (!aborted && !spin_until_ge(&sm.q_tag[qb], cur + 1, &sm.abort_flag)) aborted = true;
      __threadfence_block();
      qa = &sm.qfrag[qb][0][lane];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
#pragma unroll
        for (int gi = 0; gi < G; ++gi) qs[c][gi] = live[c] ? sm.qsum[qb][hcol[c]][gi] : 0.f;
        kap[c] = live[c] ? sm.kappa[qb][hcol[c]] : 0.f;
      }
      st.reset();
      have_seg = true;
    }
    const int slot = k % kSlots;
    const int round = k / kSlots;
    // the slot's previous chunk must have been consumed (then its fill is complete and the parity wait is exact)
    if (aborted || !spin_until_ge(&sm.released[slot], round, &sm.abort_flag) ||
        !mbar_wait(&sm.full[slot], (uint32_t)round & 1u, &sm.abort_flag)) {
      aborted = true;
      continue;
    }
    if (sm.bad[slot]) {
      poisoned = true;
    } else {
      const int j = k - seg.k0;
      // the chunk that receives the step's new token is usable once the planner warp has quantized the token into it
      if (j == seg.tail_pos && !spin_until_ge(&sm.patched[slot], round + 1, &sm.abort_flag)) { aborted = true; continue; }
      __threadfence_block();
      process_chunk<G, kBf>(sm.ring + (size_t)slot * kChunkBytes, seg.chunk_at(j) * 32, seg.lo, seg.n, g, tid, qa, qs, kap,
                       split_mask, st);
    }
    __syncwarp();
    if (lane == 0) { __threadfence_block(); *(volatile int*)&sm.released[slot] = round + 1; }
  }
  if (aborted && lane == 0) raise_flag(P.flags, Q4KV_FLAG_INTERNAL);
}

template <int G, int NW, bool kBf>
cudaError_t launch_g(const DecodeParams& P, int grid, bool pdl, cudaStream_t st) {
  static bool configured[64] = {};     // the attribute is per function and device: set it once for each
  const size_t smem = sizeof(Smem<G, NW>);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    e = cudaFuncSetAttribute(decode_mma_kernel<G, NW, kBf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3((NW + 1) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, decode_mma_kernel<G, NW, kBf>, P);
}

}  // namespace

// Number of SMs of the current device (one persistent CTA each), looked up once per device.
int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 148; }
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { (void)cudaGetLastError(); n = 148; }
    cached[dev] = n < kMaxGrid ? n : kMaxGrid;
  }
  return cached[dev];
}

bool decode_mma_supported(const Layout& y) {
  return !y.alias && y.n_rep <= 4 && ((y.D == y.Dv && (y.D == 128 || y.D == 256)) || (y.D == 192 && y.Dv == 128));
}

// the kernel counts work units in 32 bits and keeps one arrival counter per (layer of the call, agent, KV head) in
// the workspace header; chunk offsets inside the call's layers are kept in 16-byte units in 32 bits
bool decode_mma_fits(const Layout& y, int n_agents, int max_blocks, int layer_count) {
  const long long v = (long long)n_agents * layer_count;
  return layer_count >= 1 && layer_count <= kMaxLayersPerCall && v * y.Hkv * (max_blocks * 8ll) < (1ll << 30) &&
         v * y.Hkv <= kMaxTicketPairs && (unsigned long long)layer_count * y.layer_bytes < (1ull << 36);
}

// bytes behind the workspace header: one record per (layer, agent, KV head) and per CTA of the largest grid
size_t decode_mma_workspace_bytes(const Layout& y, int n_agents, int layer_count) {
  const size_t pairs = (size_t)n_agents * layer_count * y.Hkv;
  return (pairs + kMaxGrid) * y.n_rep * kRecStride(y.Dv) * sizeof(float);
}

// layer_count == 1: `windows` points at the one window.  Otherwise q, out, lse and the new rows hold layer_count
// consecutive per-layer arrays and the launch covers layers layer .. layer + layer_count - 1.
cudaError_t launch_decode_mma(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                              const int32_t* kv_lens, int max_kv_len, const int32_t* windows, int layer_count,
                              const void* q, float scale, void* out, int out_dtype, float* lse, void* ws, int32_t* flags,
                              cudaStream_t st, const void* k_new, const void* v_new) {
  if (b.n_agents <= 0 || layer_count <= 0) return cudaSuccess;
  DecodeParams P;
  P.y = y; P.pool = (const uint8_t*)pool; P.n_blocks = n_blocks; P.layer = layer; P.n_agents = b.n_agents * layer_count;
  P.n_real = b.n_agents; P.layer_count = layer_count;
  long long units = 0;
  for (int i = 0; i < kMaxLayersPerCall; ++i) {
    P.windows[i] = i < layer_count ? windows[i] : 0;
    if (i < layer_count) {
      const int span = (windows[i] > 0 && windows[i] + 32 < max_kv_len) ? windows[i] + 32 : max_kv_len;
      units += (long long)b.n_agents * y.Hkv * ((span + 31) / 32 + 1);
    }
  }
  P.max_blocks = b.max_blocks; P.len_cap = max_kv_len; P.tables = b.block_tables; P.kv_lens = kv_lens;
  P.q = (const uint16_t*)q; P.scale_log2 = scale * kLog2e;
  P.tickets = (int32_t*)ws; P.partials = (float*)((uint8_t*)ws + kWorkspaceHeaderBytes);
  P.out = out; P.out_dtype = out_dtype; P.lse = lse; P.flags = flags;
  P.k_new = (const uint16_t*)k_new; P.v_new = (const uint16_t*)v_new;
  const int n_sm = sm_count();
  const int grid = (int)(units < n_sm ? (units < 1 ? 1 : units) : n_sm);
  if (y.sb_bf16)
    return y.G == 2   ? launch_g<2, Q4KV_DECODE_WARPS_D128, true>(P, grid, true, st)
           : y.G == 3 ? launch_g<3, Q4KV_DECODE_WARPS_D128, true>(P, grid, true, st)
                      : launch_g<4, Q4KV_DECODE_WARPS_D256, true>(P, grid, true, st);
  return y.G == 2   ? launch_g<2, Q4KV_DECODE_WARPS_D128, false>(P, grid, true, st)
         : y.G == 3 ? launch_g<3, Q4KV_DECODE_WARPS_D128, false>(P, grid, true, st)
                    : launch_g<4, Q4KV_DECODE_WARPS_D256, false>(P, grid, true, st);
}

}  // namespace q4kv
