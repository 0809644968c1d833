// q4kv_quantize_append: affine 4-bit group quantization of new K/V rows, written in place
// into the agents' pool blocks (Section 3.2 format; Section 3.4 "update" step).
//
// Work unit = one "octet": the (up to) eight cache positions of one agent that share
// position/8, for one KV head.  An octet is the unit because the V codes are stored
// token-packed (eight tokens per word): one CTA owns every word it read-modify-writes.
// Eight consecutive lanes own one 64-element group (eight elements each) and reduce
// min/max with three shuffles.  Every arithmetic step is a single rounded binary32
// operation in the documented order so that codes/scales/biases are reproducible.
#include "q4kv_layout.cuh"
#include "quantize_core.cuh"

namespace q4kv {

namespace {

constexpr int kThreads = 256;

struct UnitInfo { int agent, first, cnt, row0, block; };

// Warp 0: find the (agent, octet) of unit u: agent a has ceil((pos%8 + n_a)/8) octets.  The lanes look at 32
// agents at a time, so the lengths arrive in one round trip instead of one per agent.
__device__ inline void find_unit(int u, int n_agents, int max_blocks, int n_blocks, const int32_t* __restrict__ tables,
                                 const int32_t* __restrict__ pos, const int32_t* __restrict__ new_offs, int32_t* flags,
                                 bool report_bad_len, UnitInfo* out) {
  const int lane = threadIdx.x & 31;
  int cum = 0;
  bool found = false;
  for (int base = 0; base < n_agents && !found; base += 32) {
    const int a = base + lane;
    int p = 0, r0 = 0, n = 0, octs = 0;
    bool bad_len = false;
    if (a < n_agents) {
      p = pos[a]; r0 = new_offs[a]; n = new_offs[a + 1] - r0;
      if (n > 0) {
        if (p < 0 || (long long)p + n > (long long)max_blocks * kBlockTokens) bad_len = true;
        else octs = ((p & 7) + n + 7) >> 3;
      }
    }
    if (__any_sync(0xffffffffu, bad_len) && lane == 0 && report_bad_len) raise_flag(flags, Q4KV_FLAG_BAD_LENGTH);
    int inc = octs;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const int tot = __shfl_sync(0xffffffffu, inc, 31);
    if (u < cum + tot) {
      found = true;
      const unsigned bal = __ballot_sync(0xffffffffu, cum + inc > u);
      if (lane == __ffs(bal) - 1) {
        const int uu = u - (cum + inc - octs);
        const int lo = max(p, ((p >> 3) + uu) << 3);
        const int hi = min(p + n, (((p >> 3) + uu) << 3) + 8);
        int who = a;
        const int blk = tables[(size_t)a * max_blocks + (lo >> 8)];
        if (blk < 0 || blk >= n_blocks) { raise_flag(flags, Q4KV_FLAG_BAD_BLOCK); who = -1; }
        out->agent = who; out->first = lo; out->cnt = hi - lo; out->row0 = r0 + (lo - p); out->block = blk;
      }
    }
    cum += tot;
  }
  if (!found && lane == 0) out->agent = -1;
}

// grid: (ceil(unit upper bound / M), Hkv); a CTA handles M consecutive octets.  Dynamic smem: M * 8 * Dv bytes of V
// codes (one byte per code).  M = 1 is what is launched: several octets per CTA, and one octet for all KV heads per
// CTA, both measured slower on a 8 x 1024-token phase (37 us -> 63 us for the latter): more registers per thread and
// less parallelism cost more than the shared prologue saves.  Phases of many tokens per agent take the bulk kernel
// further down; this kernel serves the appends of a few tokens per agent (3.4 us for one token of each of 5 agents).
template <int M>
__global__ void __launch_bounds__(kThreads)
quantize_append_kernel(Layout y, uint8_t* pool, int n_blocks, int layer, int n_agents, int max_blocks,
                       const int32_t* __restrict__ tables, const int32_t* __restrict__ pos,
                       const int32_t* __restrict__ new_offs, const void* __restrict__ k_new,
                       const void* __restrict__ v_new, int32_t* flags) {
  extern __shared__ uint8_t vcodes_all[];   // [M][8][Dv]
  __shared__ UnitInfo s_unit[M];
  // let the next kernel of the stream start its prologue; the unit is found from the lengths and block tables (inputs
  // that no kernel writes) while the preceding kernels drain, and the wait comes before the new rows and the pool
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x < 32) {
    for (int r = 0; r < M; ++r)
      find_unit(blockIdx.x * M + r, n_agents, max_blocks, n_blocks, tables, pos, new_offs, flags,
                blockIdx.x == 0 && blockIdx.y == 0 && r == 0, &s_unit[r]);
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int hk = blockIdx.y;
  const int kw = y.D / 8, vw = y.alias ? 0 : y.Dv / 8;
  const int n_items = 8 * (kw + vw);

  // ---- K and V rows in one sweep: items (tensor, token i, word w), eight lanes per group.  K words and
  // scale/bias pairs go straight to the pool; V codes go to shared memory as bytes for the transposition. ----
  for (int base = 0; base < n_items; base += kThreads) {
    const int idx = base + threadIdx.x;
    const bool is_v = idx >= 8 * kw;
    const int j = is_v ? idx - 8 * kw : idx, ww = is_v ? vw : kw;
    const int i = j / (ww > 0 ? ww : 1), w = j % (ww > 0 ? ww : 1);
    float x[M][8];
    bool live[M];
#pragma unroll
    for (int r = 0; r < M; ++r) {
      const UnitInfo un = s_unit[r];
      live[r] = un.agent >= 0 && idx < n_items && i < un.cnt;
      if (live[r]) {
        if (is_v) load_eight_bf16(v_new, ((size_t)(un.row0 + i) * y.Hkv + hk) * y.Dv + 8 * w, x[r]);
        else load_eight_bf16(k_new, ((size_t)(un.row0 + i) * y.Hkv + hk) * y.D + 8 * w, x[r]);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) x[r][e] = 0.f;
      }
    }
#pragma unroll
    for (int r = 0; r < M; ++r) {
      const QuantOut o = quantize_eight(x[r], y.sb_bf16 != 0);
      if (!live[r]) continue;
      const UnitInfo un = s_unit[r];
      const int slot0 = un.first & 255;                 // the octet lies inside one 32-token chunk
      uint8_t* chunk = head_block(pool, y, layer, un.block, hk) + (size_t)(slot0 >> 5) * y.chunk_bytes;
      const int tau = (slot0 & 31) + i;
      if (is_v) {
        uint8_t* vcodes = vcodes_all + (size_t)r * 8 * y.Dv;
#pragma unroll
        for (int e = 0; e < 8; ++e) vcodes[i * y.Dv + 8 * w + e] = (o.word >> (4 * e)) & 15u;
        if ((w & 7) == 0) reinterpret_cast<uint32_t*>(chunk + y.off_vsb)[sb_offset(tau, w >> 3, y.Gv)] = o.sb;
      } else {
        reinterpret_cast<uint32_t*>(chunk + y.off_kc)[k_word_offset(tau, w, y.G)] = o.word;
        if ((w & 7) == 0) reinterpret_cast<uint32_t*>(chunk + y.off_ksb)[sb_offset(tau, w >> 3, y.G)] = o.sb;
      }
    }
  }
  if (y.alias) return;
  __syncthreads();
  // ---- token-packed V words: one word = one head-dim element of the octet's 8 positions ----
#pragma unroll
  for (int r = 0; r < M; ++r) {
    const UnitInfo un = s_unit[r];
    if (un.agent < 0) continue;
    const uint8_t* vcodes = vcodes_all + (size_t)r * 8 * y.Dv;
    const int slot0 = un.first & 255, tau0 = slot0 & 31;
    uint8_t* chunk = head_block(pool, y, layer, un.block, hk) + (size_t)(slot0 >> 5) * y.chunk_bytes;
    const int k0 = un.first & 7;              // nibble of the first new token inside the word
    uint32_t mask = 0;
    for (int i = 0; i < un.cnt; ++i) mask |= 15u << (4 * (k0 + i));
    uint32_t* vc = reinterpret_cast<uint32_t*>(chunk + y.off_vc);
    for (int d = threadIdx.x; d < y.Dv; d += kThreads) {
      uint32_t bits = 0;
      for (int i = 0; i < un.cnt; ++i) bits |= (uint32_t)vcodes[i * y.Dv + d] << (4 * (k0 + i));
      const int wi = v_word_offset(tau0 >> 3, d);
      vc[wi] = (mask == 0xffffffffu) ? bits : ((vc[wi] & ~mask) | bits);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Bulk form (a prefill phase: many new tokens per agent).  One warp owns one (32-token chunk, KV head) unit and walks
// its items -- (octet of eight positions, pass of four groups: K groups first, then V groups) -- with the loads of the
// next item in flight while the current one is quantized.  Within an item a lane owns one of the eight positions and
// one 64-element group: it loads its 64 elements as eight 16-byte words, takes minimum and maximum with packed bf16
// instructions (no cross-lane step at all), and quantizes them: the quotient as t * (1/scale), rounded by adding
// 1.5 * 2^23 (the code is then in the low bits), and only a quotient within 4e-6 of a tie goes through the division
// itself, so that the codes equal those of the fixed sequence bit for bit.  V words are first exchanged between the
// eight lanes of a group (an 8 x 8 transposition of words by twelve shuffles), which leaves in each lane the
// 8 positions x 8 elements block of nibbles that an in-register transposition turns into eight token-packed words.
// The chunk is assembled in shared memory and stored as whole 16-byte pieces; a chunk that the phase fills only in
// part (an unaligned start or end) starts from its present bytes.
// Measured on 8 x 1024 tokens (43 MB): 20.1 us, bound by instruction issue (about 1230 warp instructions per item of
// 32 x 64 elements at 0.5 issued per scheduler and clock); the same time with one warp per octet and direct stores.
// ---------------------------------------------------------------------------------------------
__device__ inline void transpose_nibbles_8x8_regs(uint32_t (&r)[8]) {
  // rows = registers, columns = nibbles: three rounds of block swaps
#pragma unroll
  for (int s = 1; s < 8; s <<= 1) {
    const uint32_t m = s == 1 ? 0x0F0F0F0Fu : s == 2 ? 0x00FF00FFu : 0x0000FFFFu;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (t & s) continue;
      const uint32_t x = ((r[t] >> (4 * s)) ^ r[t + s]) & m;
      r[t + s] ^= x;
      r[t] ^= x << (4 * s);
    }
  }
}

// Code of one element by the division itself (the rare element whose quotient is within a few ulps of a tie).  A call, so
// that the compiler keeps the division out of the common path.
__device__ __noinline__ float exact_code(float x, float bf, float sf) {
  return fminf(rintf(__fdiv_rn(__fsub_rn(x, bf), sf)), 15.0f);
}

// Unit of the bulk kernel: one 32-token chunk of one agent's new range (up to four octets, all in one pool block).
struct ChunkUnit { int agent, p, n, r0, chunk, block; };

// Warp-wide: find the (agent, chunk) of unit u; agent a has chunk(p + n - 1) - chunk(p) + 1 units.
__device__ inline void find_chunk_unit(int u, int n_agents, int max_blocks, int n_blocks, const int32_t* __restrict__ tables,
                                       const int32_t* __restrict__ pos, const int32_t* __restrict__ new_offs, int32_t* flags,
                                       bool report_bad_len, ChunkUnit* out) {
  const int lane = threadIdx.x & 31;
  int cum = 0;
  bool found = false;
  for (int base = 0; base < n_agents && !found; base += 32) {
    const int a = base + lane;
    int p = 0, r0 = 0, n = 0, cnt = 0;
    bool bad_len = false;
    if (a < n_agents) {
      p = pos[a]; r0 = new_offs[a]; n = new_offs[a + 1] - r0;
      if (n > 0) {
        if (p < 0 || (long long)p + n > (long long)max_blocks * kBlockTokens) bad_len = true;
        else cnt = ((p + n - 1) >> 5) - (p >> 5) + 1;
      }
    }
    if (__any_sync(0xffffffffu, bad_len) && lane == 0 && report_bad_len) raise_flag(flags, Q4KV_FLAG_BAD_LENGTH);
    int inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const int tot = __shfl_sync(0xffffffffu, inc, 31);
    if (u < cum + tot) {
      found = true;
      const unsigned bal = __ballot_sync(0xffffffffu, cum + inc > u);
      if (lane == __ffs(bal) - 1) {
        const int c = (p >> 5) + (u - (cum + inc - cnt));
        int who = a;
        const int blk = tables[(size_t)a * max_blocks + (c >> 3)];
        if (blk < 0 || blk >= n_blocks) { raise_flag(flags, Q4KV_FLAG_BAD_BLOCK); who = -1; }
        out->agent = who; out->p = p; out->n = n; out->r0 = r0; out->chunk = c; out->block = blk;
      }
    }
    cum += tot;
  }
  if (!found && lane == 0) out->agent = -1;
}

// One warp owns one (chunk, KV head) unit and walks its items -- (octet, pass of four groups) -- with the loads of
// the next item in flight while the current one is quantized.
__global__ void __launch_bounds__(kThreads, 2)
quantize_append_bulk_kernel(Layout y, uint8_t* pool, int n_blocks, int layer, int n_agents, int max_blocks,
                            const int32_t* __restrict__ tables, const int32_t* __restrict__ pos,
                            const int32_t* __restrict__ new_offs, const uint16_t* __restrict__ k_new,
                            const uint16_t* __restrict__ v_new, int32_t* flags, int units) {
  __shared__ ChunkUnit s_unit[kThreads / 32];
  extern __shared__ __align__(16) uint8_t stage_all[];  // one chunk per warp
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (kThreads / 32) + warp;
  const int u = gw / y.Hkv, hk = gw - u * y.Hkv;
  if (u >= units) return;
  find_chunk_unit(u, n_agents, max_blocks, n_blocks, tables, pos, new_offs, flags, gw == 0, &s_unit[warp]);
  __syncwarp();
  const ChunkUnit un = s_unit[warp];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (un.agent < 0) return;

  const int s = lane & 7, gq0 = lane >> 3;             // position slot inside an octet, group inside a pass
  const int c0 = un.chunk << 5;                          // first cache position of the chunk
  const int lo = max(un.p, c0), hi = min(un.p + un.n, c0 + 32);
  const int o_first = (lo - c0) >> 3, o_last = (hi - 1 - c0) >> 3;
  // The chunk is put together in shared memory and leaves as whole 16-byte pieces (the words of a token are scattered
  // over the chunk: stored one by one they would reach L2 as a million and a half partial sectors per phase).  A
  // chunk that this phase fills only in part starts from its present bytes; this warp is its only writer.
  uint8_t* gchunk = head_block(pool, y, layer, un.block, hk) + (size_t)(un.chunk & 7) * y.chunk_bytes;
  uint8_t* chunk = stage_all + (size_t)warp * y.chunk_bytes;
  const int n16 = y.chunk_bytes / 16;
  if (lo != c0 || hi != c0 + 32) {
    for (int q = lane; q < n16; q += 32) reinterpret_cast<uint4*>(chunk)[q] = reinterpret_cast<const uint4*>(gchunk)[q];
    __syncwarp();
  }
  const int n_groups = y.G + (y.alias ? 0 : y.Gv);
  const int n_pass = (n_groups + 3) >> 2;
  const int n_items = (o_last - o_first + 1) * n_pass;
  constexpr float kMagic = 12582912.0f;                  // 1.5 * 2^23: (q + kMagic) - kMagic is q rounded to nearest even
  // t * inv is within 2 ulps (2e-6 at q < 16) of the quotient the fixed sequence rounds: beyond 4e-6 of a tie both round
  // to the same code
  constexpr float kTieZone = 0.499996f;

  // item t: octet o_first + t / n_pass of the chunk, groups 4 * (t % n_pass) .. + 3
  auto load_item = [&](int t, uint4 (&raw)[8]) {
    const int o = o_first + t / n_pass, pass = t - (t / n_pass) * n_pass;
    const int first = max(lo, c0 + 8 * o), cnt = min(hi, c0 + 8 * o + 8) - first;
    const int i = s - (first & 7);
    const int gq = pass * 4 + gq0;
    const bool is_v = gq >= y.G;
    const int gi = is_v ? gq - y.G : gq;
    if (gq < n_groups && i >= 0 && i < cnt) {
      const size_t row = (size_t)(un.r0 + (first - un.p) + i) * y.Hkv + hk;
      const uint16_t* src = is_v ? v_new + row * y.Dv + 64 * gi : k_new + row * y.D + 64 * gi;
#pragma unroll
      for (int j = 0; j < 8; ++j) raw[j] = __ldg(reinterpret_cast<const uint4*>(src) + j);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) raw[j] = make_uint4(0u, 0u, 0u, 0u);
    }
  };

  uint4 raw[8], nxt[8];
  load_item(0, raw);
  for (int t = 0; t < n_items; ++t) {
    if (t + 1 < n_items) load_item(t + 1, nxt);
    const int o = o_first + t / n_pass, pass = t - (t / n_pass) * n_pass;
    const int first = max(lo, c0 + 8 * o), cnt = min(hi, c0 + 8 * o + 8) - first;
    const int k0 = first & 7;
    const int i = s - k0;                                // this lane's token of the octet
    const bool tok = i >= 0 && i < cnt;
    const int tau = 8 * o + s;                           // chunk token of this lane's position
    const uint32_t nib_mask = cnt == 8 ? 0xFFFFFFFFu : (((1u << (4 * cnt)) - 1u) << (4 * k0));
    const int gq = pass * 4 + gq0;
    const bool has = gq < n_groups;
    const bool is_v = has && gq >= y.G;
    const int gi = is_v ? gq - y.G : gq;
    const bool active = has && tok;
    // minimum and maximum of the 64 elements on packed bf16 (values are exact, so this is the binary32 result)
    __nv_bfloat162 mn2 = *reinterpret_cast<const __nv_bfloat162*>(&raw[0].x), mx2 = mn2;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t wv[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&wv[e]);
        mn2 = __hmin2(mn2, v);
        mx2 = __hmax2(mx2, v);
      }
    }
    const uint32_t mnb = *reinterpret_cast<const uint32_t*>(&mn2), mxb = *reinterpret_cast<const uint32_t*>(&mx2);
    const float mn = fminf(__uint_as_float(mnb << 16), __uint_as_float(mnb & 0xffff0000u));
    const float mx = fmaxf(__uint_as_float(mxb << 16), __uint_as_float(mxb & 0xffff0000u));
    const GroupScale gs = group_scale(mn, mx, y.sb_bf16 != 0);
    uint32_t cw[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) cw[j] = 0u;
    if (gs.sf != 0.0f) {
      const float inv = __frcp_rn(gs.sf);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t wv[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
        // t = x - bias, q = t / scale (as t * inv), c = q rounded to nearest even by adding and subtracting 1.5 * 2^23;
        // q <= 15 + a few ulps by construction of the scale, so no clamp is needed.  The eight codes are assembled in
        // floating point (two exact 16-bit halves) instead of by shifts.
        float c[8], far = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x = (e & 1) ? __uint_as_float(wv[e >> 1] & 0xffff0000u) : __uint_as_float(wv[e >> 1] << 16);
          const float q = __fmul_rn(__fsub_rn(x, gs.bf), inv);
          c[e] = __fsub_rn(__fadd_rn(q, kMagic), kMagic);
          far = fmaxf(far, fabsf(__fsub_rn(q, c[e])));
        }
        if (far > kTieZone) {                            // rare: some quotient is too close to a tie for t * inv to decide
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float x = (e & 1) ? __uint_as_float(wv[e >> 1] & 0xffff0000u) : __uint_as_float(wv[e >> 1] << 16);
            const float q = __fmul_rn(__fsub_rn(x, gs.bf), inv);
            if (fabsf(__fsub_rn(q, c[e])) > kTieZone) c[e] = exact_code(x, gs.bf, gs.sf);
          }
        }
        const float lo4 = fmaf(fmaf(fmaf(c[3], 16.f, c[2]), 16.f, c[1]), 16.f, c[0]);
        const float hi4 = fmaf(fmaf(fmaf(c[7], 16.f, c[6]), 16.f, c[5]), 16.f, c[4]);
        cw[j] = __byte_perm(__float_as_uint(lo4 + 8388608.0f), __float_as_uint(hi4 + 8388608.0f), 0x5410);
      }
    }
    const uint32_t sb = gs.hs | (gs.hb << 16);
    if (active && !is_v) {
      // words w = 8 gi + 4 i2 + t sit in 16-byte pieces of four (group, half) words: this lane's pair is 8 bytes
      uint32_t* kc = reinterpret_cast<uint32_t*>(chunk + y.off_kc);
#pragma unroll
      for (int w = 0; w < 4; ++w)
        *reinterpret_cast<uint2*>(kc + k_word_offset(tau, 8 * gi + w, y.G)) = make_uint2(cw[w], cw[4 + w]);
      reinterpret_cast<uint32_t*>(chunk + y.off_ksb)[sb_offset(tau, gi, y.G)] = sb;
    }
    if (pass * 4 + 3 >= y.G) {                           // not a pass of K groups only (warp-uniform)
      if (active && is_v) reinterpret_cast<uint32_t*>(chunk + y.off_vsb)[sb_offset(tau, gi, y.Gv)] = sb;
      // 8 x 8 transposition of words between the eight lanes of a group: afterwards lane s holds, in cw[w], word s
      // (elements 8s .. 8s+7 of the group) of position w
#pragma unroll
      for (int b = 4; b > 0; b >>= 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j & b) continue;
          const uint32_t send = (s & b) ? cw[j] : cw[j | b];
          const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, b);
          if (s & b) cw[j] = recv; else cw[j | b] = recv;
        }
      }
      transpose_nibbles_8x8_regs(cw);                    // cw[e]: element 8s + e of the group, nibble w = position w
      if (is_v) {
        uint32_t* vc = reinterpret_cast<uint32_t*>(chunk + y.off_vc);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          uint32_t* at = vc + v_word_offset(o, 64 * gi + 8 * s + e);
          *at = nib_mask == 0xFFFFFFFFu ? cw[e] : ((*at & ~nib_mask) | (cw[e] & nib_mask));
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) raw[j] = nxt[j];
  }
  __syncwarp();
  for (int q = lane; q < n16; q += 32) reinterpret_cast<uint4*>(gchunk)[q] = reinterpret_cast<const uint4*>(chunk)[q];
}

template <int M>
cudaError_t launch_m(const Layout& y, uint8_t* pool, int n_blocks, int layer, const q4kv_batch& b, const int32_t* pos,
                     const int32_t* new_offs, int units, const void* k_new, const void* v_new, int32_t* flags,
                     cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((units + M - 1) / M, y.Hkv);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = y.alias ? 0 : (size_t)M * 8 * y.Dv;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, quantize_append_kernel<M>, y, pool, n_blocks, layer, b.n_agents, b.max_blocks,
                            b.block_tables, pos, new_offs, k_new, v_new, flags);
}

}  // namespace

cudaError_t launch_quantize_append(const Layout& y, void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                   const int32_t* pos, const int32_t* new_offs, int total_new,
                                   const void* k_new, const void* v_new, int32_t* flags, cudaStream_t st) {
  if (total_new <= 0 || b.n_agents <= 0) return cudaSuccess;
  const int units = total_new / 8 + 2 * b.n_agents;        // >= sum over agents of ceil((pos%8+n)/8)
  if (total_new >= 8 * b.n_agents && (size_t)(kThreads / 32) * y.chunk_bytes <= 112 * 1024) {
    // a phase of many tokens per agent: one warp per (32-token chunk, KV head)
    const int chunk_units = total_new / 32 + 2 * b.n_agents;   // >= sum over agents of the chunks their new range touches
    const long long warps = (long long)chunk_units * y.Hkv;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((warps + kThreads / 32 - 1) / (kThreads / 32)));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)(kThreads / 32) * y.chunk_bytes;
    cfg.stream = st;
    static bool configured[64] = {};     // the attribute is per function and device: set it once for each
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
      e = cudaFuncSetAttribute(quantize_append_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024);
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, quantize_append_bulk_kernel, y, (uint8_t*)pool, n_blocks, layer, b.n_agents,
                              b.max_blocks, b.block_tables, pos, new_offs, (const uint16_t*)k_new,
                              (const uint16_t*)v_new, flags, chunk_units);
  }
  return launch_m<1>(y, (uint8_t*)pool, n_blocks, layer, b, pos, new_offs, units, k_new, v_new, flags, st);
}

}  // namespace q4kv
