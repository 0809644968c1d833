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
// less parallelism cost more than the shared prologue saves.  One warp per octet with its loads batched ahead of the
// arithmetic: 35 us on that phase, but 1.5-2 us slower on the single-token launches of a decode step.  The phase is
// bound by instruction issue (about 230 instructions per eight elements), not by bytes in flight.
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
      const QuantOut o = quantize_eight(x[r]);
      if (!live[r]) continue;
      const UnitInfo un = s_unit[r];
      const int slot0 = un.first & 255;                 // the octet lies inside one 32-token chunk
      uint8_t* chunk = head_block(pool, y, layer, un.block, hk) + (size_t)(slot0 >> 5) * y.chunk_bytes;
      const int tau = (slot0 & 31) + i;
      if (is_v) {
        uint8_t* vcodes = vcodes_all + (size_t)r * 8 * y.Dv;
#pragma unroll
        for (int e = 0; e < 8; ++e) vcodes[i * y.Dv + 8 * w + e] = (o.word >> (4 * e)) & 15u;
        if ((w & 7) == 0) reinterpret_cast<__half2*>(chunk + y.off_vsb)[sb_offset(tau, w >> 3, y.Gv)] = o.sb;
      } else {
        reinterpret_cast<uint32_t*>(chunk + y.off_kc)[k_word_offset(tau, w, y.G)] = o.word;
        if ((w & 7) == 0) reinterpret_cast<__half2*>(chunk + y.off_ksb)[sb_offset(tau, w >> 3, y.G)] = o.sb;
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
  return launch_m<1>(y, (uint8_t*)pool, n_blocks, layer, b, pos, new_offs, units, k_new, v_new, flags, st);
}

}  // namespace q4kv
