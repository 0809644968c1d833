// Generic Q4 attention kernels (any supported spec): decode (one query per agent) and
// chunked prefill (a block of causal queries per agent) over the in-place Q4 cache, with
// split-K partials and a merge kernel.  Sections 3.4-3.6: fused attention on Q4 tensors,
// GQA head mapping, sliding-window layers, asymmetric / aliased value dims.
//
// This is the shape-agnostic CUDA-core path: correct for every spec the library accepts and
// the fallback for shapes without a tensor-core specialisation.  One CTA handles one
// (query item, query head, key split); a warp walks octets (8 tokens), dequantizes K rows into
// a shared tile, takes the scores from registers, keeps an online softmax (base-2) and
// accumulates P.V from the token-packed V words (or from the K tile when V aliases K).
#include "q4kv_layout.cuh"

namespace q4kv {

namespace {

// a (scale, bias) pair of the cache as two binary32 numbers: binary16 or bfloat16 halves
__device__ inline float2 sb_pair(uint32_t u, bool bf16) {
  if (bf16) return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxDvPerLane = 16;      // Dv <= 512
constexpr float kLog2e = 1.4426950408889634f;

struct ItemInfo { int agent, q_row, pos_end, lo; };   // keys [lo, pos_end)

// Decode: item = agent.  Prefill: item = global query row; agent found by scanning q_offs.
// len_cap: the host's bound on every length (at most max_blocks * 256); the key splits cover exactly that many keys
__device__ inline bool locate_item(int item, int n_agents, const int32_t* kv_lens, const int32_t* q_offs,
                                   int window, int len_cap, int32_t* flags, ItemInfo& it) {
  int a, pos_end;
  if (q_offs == nullptr) {
    a = item;
    pos_end = kv_lens[a];
  } else {
    a = 0;
    while (a + 1 < n_agents && item >= q_offs[a + 1]) ++a;
    const int q_len = q_offs[a + 1] - q_offs[a];
    const int n = kv_lens[a];
    if (item >= q_offs[n_agents] || q_len > n) {
      raise_flag(flags, Q4KV_FLAG_BAD_LENGTH);
      it.agent = a; it.q_row = item; it.pos_end = -1; it.lo = 0;
      return false;
    }
    pos_end = n - q_len + (item - q_offs[a]) + 1;
  }
  it.agent = a; it.q_row = item;
  const int n_all = kv_lens[a];
  if (n_all < 0 || n_all > len_cap) {
    raise_flag(flags, Q4KV_FLAG_BAD_LENGTH);
    it.pos_end = -1; it.lo = 0;
    return false;
  }
  it.pos_end = pos_end;
  it.lo = window > 0 ? max(0, pos_end - window) : 0;
  return true;
}

// grid: (n_items, Hq, n_splits); dynamic smem: D floats (q) + kWarps * 8 * D floats (K tiles)
//       + kWarps * (Dv + 2) floats (cross-warp merge)
__global__ void __launch_bounds__(kThreads)
attn_generic_kernel(Layout y, const uint8_t* __restrict__ pool, int n_blocks, int layer, int n_agents,
                    int max_blocks, int len_cap, const int32_t* __restrict__ tables, const int32_t* __restrict__ kv_lens,
                    const int32_t* __restrict__ q_offs, int window, const uint16_t* __restrict__ q,
                    float scale_log2, int n_splits, int split_tokens,
                    float* __restrict__ partials, void* __restrict__ out, int out_dtype,
                    float* __restrict__ lse, int32_t* flags) {
  extern __shared__ float smem[];
  float* sq = smem;                                  // [D]
  float* stile = sq + y.D;                           // [kWarps][8][D]
  float* smerge = stile + kWarps * 8 * y.D;          // [kWarps][Dv + 2]
  const int item = blockIdx.x, h = blockIdx.y, split = blockIdx.z;
  const int hk = h / y.n_rep;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int D = y.D, Dv = y.Dv, G = y.G;
  const int nd = Dv / 32;

  ItemInfo it;
  const bool ok = locate_item(item, n_agents, kv_lens, q_offs, window, len_cap, flags, it);
  const size_t out_index = ((size_t)it.q_row * y.Hq + h) * Dv;
  float* part = partials + (((size_t)item * y.Hq + h) * n_splits + split) * (Dv + 2);

  // this CTA's key range
  const int base = it.lo & ~7;
  int t0 = base + split * split_tokens, t1 = min(t0 + split_tokens, it.pos_end);
  if (!ok || it.pos_end <= it.lo) { t0 = 0; t1 = 0; }
  bool bad_block = false;

  for (int d = threadIdx.x; d < D; d += kThreads)
    sq[d] = bf16_bits_to_float(q[((size_t)it.q_row * y.Hq + h) * D + d]) * scale_log2;
  __syncthreads();

  float m = -INFINITY, l = 0.f, acc[kMaxDvPerLane];
#pragma unroll
  for (int i = 0; i < kMaxDvPerLane; ++i) acc[i] = 0.f;
  float* tile = stile + warp * 8 * D;
  const int k = lane >> 2, t = lane & 3;

  for (int o0 = t0 + 8 * warp; o0 < t1; o0 += 8 * kWarps) {
    // one octet [o0, o0+8) lies inside one block
    const int blk = tables[(size_t)it.agent * max_blocks + (o0 >> 8)];
    if (blk < 0 || blk >= n_blocks) { bad_block = true; break; }
    const int slot0 = o0 & 255;
    const uint8_t* chunk = head_block(pool, y, layer, blk, hk) + (size_t)(slot0 >> 5) * y.chunk_bytes;
    const int tau0 = slot0 & 31;
    const int tok = o0 + k;
    const bool valid = tok >= it.lo && tok < t1;
    // ---- dequantize this lane's quarter of row k, score from registers ----
    float s = 0.f;
    {
      const uint32_t* kc = reinterpret_cast<const uint32_t*>(chunk + y.off_kc);
      const uint32_t* ksb = reinterpret_cast<const uint32_t*>(chunk + y.off_ksb);
      for (int p = 0; p < 2 * G; ++p) {
        const int gi = p >> 1, i2 = p & 1;
        const int w = 8 * gi + 4 * i2 + t;
        float sc = 0.f, bi = 0.f;
        uint32_t word = 0;
        if (valid) {
          const float2 f = sb_pair(ksb[sb_offset(tau0 + k, gi, G)], y.sb_bf16 != 0);
          sc = f.x; bi = f.y;
          word = kc[k_word_offset(tau0 + k, w, G)];
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x = valid ? fmaf((float)((word >> (4 * e)) & 15u), sc, bi) : 0.f;
          tile[k * D + 8 * w + e] = x;
          s = fmaf(x, sq[8 * w + e], s);
        }
      }
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if (!valid) s = -INFINITY;
    float mx = s;
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
    const float m_new = fmaxf(m, mx);
    // the octet always holds at least one valid token here, so m_new is finite
    const float corr = exp2f(m - m_new);
    const float p_me = valid ? exp2f(s - m_new) : 0.f;
    float psum = (t == 0) ? p_me : 0.f;
    psum += __shfl_xor_sync(0xffffffffu, psum, 4);
    psum += __shfl_xor_sync(0xffffffffu, psum, 8);
    psum += __shfl_xor_sync(0xffffffffu, psum, 16);
    psum += __shfl_xor_sync(0xffffffffu, psum, 1);
    psum += __shfl_xor_sync(0xffffffffu, psum, 2);
    l = l * corr + psum;
    m = m_new;
    float p[8];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) p[kk] = __shfl_sync(0xffffffffu, p_me, 4 * kk);
    __syncwarp();
    // ---- P.V ----
    if (y.alias) {
#pragma unroll
      for (int i = 0; i < kMaxDvPerLane; ++i) {
        if (i >= nd) break;
        const int d = lane + 32 * i;
        float a = acc[i] * corr;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) a = fmaf(p[kk], tile[kk * D + d], a);
        acc[i] = a;
      }
    } else {
      const uint32_t* vc = reinterpret_cast<const uint32_t*>(chunk + y.off_vc);
      const uint32_t* vsb = reinterpret_cast<const uint32_t*>(chunk + y.off_vsb);
#pragma unroll
      for (int i = 0; i < kMaxDvPerLane; ++i) {
        if (i >= nd) break;
        const int d = lane + 32 * i, gi = d >> 6;
        const uint32_t word = vc[v_word_offset(tau0 >> 3, d)];
        float a = acc[i] * corr;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          if (p[kk] != 0.f) {     // invalid tokens may hold garbage scale bits
            const float2 f = sb_pair(vsb[sb_offset(tau0 + kk, gi, y.Gv)], y.sb_bf16 != 0);
            a = fmaf(p[kk], fmaf((float)((word >> (4 * kk)) & 15u), f.x, f.y), a);
          }
        }
        acc[i] = a;
      }
    }
    __syncwarp();
  }

  // ---- cross-warp merge ----
  float* mine = smerge + warp * (Dv + 2);
  if (lane == 0) { mine[Dv] = m; mine[Dv + 1] = l; }
#pragma unroll
  for (int i = 0; i < kMaxDvPerLane; ++i)
    if (i < nd) mine[lane + 32 * i] = acc[i];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  if (bad_block && lane == 0) s_bad = 1;
  __syncthreads();
  if (s_bad) {
    if (threadIdx.x == 0) raise_flag(flags, Q4KV_FLAG_BAD_BLOCK);
  }
  float M = -INFINITY;
  for (int w = 0; w < kWarps; ++w) M = fmaxf(M, smerge[w * (Dv + 2) + Dv]);
  float Lsum = 0.f;
  float wgt[kWarps];
  for (int w = 0; w < kWarps; ++w) {
    const float mw = smerge[w * (Dv + 2) + Dv];
    wgt[w] = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
    Lsum += wgt[w] * smerge[w * (Dv + 2) + Dv + 1];
  }
  if (s_bad) { M = -INFINITY; Lsum = -1.f; }   // negative sum = poisoned partial: the merge writes zeros
  for (int d = threadIdx.x; d < Dv; d += kThreads) {
    float a = 0.f;
    for (int w = 0; w < kWarps; ++w) a += wgt[w] * smerge[w * (Dv + 2) + d];
    if (s_bad) a = 0.f;
    if (n_splits > 1) {
      part[d] = a;
    } else {
      const float o = Lsum > 0.f ? a / Lsum : 0.f;
      if (out_dtype == Q4KV_OUT_BF16) reinterpret_cast<__nv_bfloat16*>(out)[out_index + d] = __float2bfloat16_rn(o);
      else reinterpret_cast<float*>(out)[out_index + d] = o;
    }
  }
  if (threadIdx.x == 0) {
    if (n_splits > 1) { part[Dv] = M; part[Dv + 1] = Lsum; }
    else if (lse) lse[(size_t)it.q_row * y.Hq + h] = Lsum > 0.f ? (M + log2f(Lsum)) / kLog2e : -INFINITY;
  }
}

// grid: (Hq, n_items); combines the split partials of one (item, head)
__global__ void __launch_bounds__(128)
merge_splits_kernel(int Hq, int Dv, int n_splits, const float* __restrict__ partials, void* __restrict__ out,
                    int out_dtype, float* __restrict__ lse) {
  const int h = blockIdx.x, item = blockIdx.y;
  const float* part = partials + (((size_t)item * Hq + h) * n_splits) * (Dv + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part[(size_t)s * (Dv + 2) + Dv]);
  float Lsum = 0.f;
  bool poisoned = false;
  for (int s = 0; s < n_splits; ++s) {
    const float ms = part[(size_t)s * (Dv + 2) + Dv];
    if (part[(size_t)s * (Dv + 2) + Dv + 1] < 0.f) poisoned = true;
    if (ms != -INFINITY) Lsum += exp2f(ms - M) * part[(size_t)s * (Dv + 2) + Dv + 1];
  }
  if (poisoned) Lsum = 0.f;
  const size_t out_index = ((size_t)item * Hq + h) * Dv;
  for (int d = threadIdx.x; d < Dv; d += blockDim.x) {
    float a = 0.f;
    for (int s = 0; s < n_splits; ++s) {
      const float ms = part[(size_t)s * (Dv + 2) + Dv];
      if (ms != -INFINITY) a += exp2f(ms - M) * part[(size_t)s * (Dv + 2) + d];
    }
    const float o = Lsum > 0.f ? a / Lsum : 0.f;
    if (out_dtype == Q4KV_OUT_BF16) reinterpret_cast<__nv_bfloat16*>(out)[out_index + d] = __float2bfloat16_rn(o);
    else reinterpret_cast<float*>(out)[out_index + d] = o;
  }
  if (threadIdx.x == 0 && lse) lse[(size_t)item * Hq + h] = Lsum > 0.f ? (M + log2f(Lsum)) / kLog2e : -INFINITY;
}

}  // namespace

DecodePlan plan_decode(const Layout& y, int n_agents, int max_kv_len, int window) {
  // keys one query can touch (the window start is rounded down to a multiple of 8)
  const int span = (window > 0 && window + 8 < max_kv_len) ? window + 8 : max_kv_len;
  const int ctas = n_agents * y.Hq;
  int n_splits = (4 * sm_count() + ctas - 1) / ctas;
  const int max_splits = (span + 255) / 256;
  if (n_splits > max_splits) n_splits = max_splits;
  if (n_splits < 1) n_splits = 1;
  int st = (span + n_splits - 1) / n_splits;
  st = (st + 63) & ~63;
  if (st < 64) st = 64;
  n_splits = (span + st - 1) / st;
  if (n_splits < 1) n_splits = 1;
  DecodePlan p;
  p.n_splits = n_splits;
  p.split_tokens = st;
  return p;
}

cudaError_t launch_attention_generic(const Layout& y, const void* pool, int n_blocks, int layer, const q4kv_batch& b,
                                     const int32_t* kv_lens, const int32_t* q_offs, int total_q, int max_q_len,
                                     int max_kv_len, int window, const void* q, float scale, void* out,
                                     int out_dtype, float* lse, void* ws, int32_t* flags, cudaStream_t st) {
  (void)max_q_len;
  const bool prefill = q_offs != nullptr;
  const int items = prefill ? total_q : b.n_agents;
  if (items <= 0) return cudaSuccess;
  DecodePlan plan;
  if (prefill) { plan.n_splits = 1; plan.split_tokens = (max_kv_len + 63) & ~63; if (plan.split_tokens < 64) plan.split_tokens = 64; }
  else plan = plan_decode(y, b.n_agents, max_kv_len, window);
  const size_t smem = sizeof(float) * ((size_t)y.D + (size_t)kWarps * 8 * y.D + (size_t)kWarps * (y.Dv + 2));
  cudaError_t e = cudaFuncSetAttribute(attn_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  {
    dim3 grid(items, y.Hq, plan.n_splits);
    attn_generic_kernel<<<grid, kThreads, smem, st>>>(
        y, (const uint8_t*)pool, n_blocks, layer, b.n_agents, b.max_blocks, max_kv_len, b.block_tables, kv_lens, q_offs,
        window, (const uint16_t*)q, scale * kLog2e, plan.n_splits, plan.split_tokens, (float*)ws, out, out_dtype,
        lse, flags);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (plan.n_splits > 1) {
    dim3 grid(y.Hq, items);
    merge_splits_kernel<<<grid, 128, 0, st>>>(y.Hq, y.Dv, plan.n_splits, (const float*)ws, out, out_dtype, lse);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace q4kv
