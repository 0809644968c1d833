// C ABI of libq4kv.so: host-side validation, sizing and dispatch.  See include/q4kv.h for
// the contract of every entry point.
#include "q4kv_layout.cuh"

using namespace q4kv;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_spec(const q4kv_spec* s) {
  if (!s) return Q4KV_EINVAL;
  if (s->n_layers <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->d_qk <= 0 || s->d_v <= 0) return Q4KV_EINVAL;
  if (s->group != 64 || s->block_tokens != 256 || (s->sb_dtype != 0 && s->sb_dtype != 1)) return Q4KV_EUNSUPPORTED;
  if (s->exact_products != 0 && s->exact_products != 1) return Q4KV_EINVAL;
  if (s->d_qk % 64 || s->d_v % 64 || s->n_q_heads % s->n_kv_heads) return Q4KV_EUNSUPPORTED;
  if (s->d_qk > 1024 || s->d_v > 512) return Q4KV_EUNSUPPORTED;
  if (s->v_aliases_k && s->d_v > s->d_qk) return Q4KV_EUNSUPPORTED;
  return Q4KV_OK;
}

int check_batch(const q4kv_batch* b) {
  if (!b || b->n_agents < 0 || b->max_blocks <= 0) return Q4KV_EINVAL;
  if (b->n_agents > 0 && !b->block_tables) return Q4KV_EINVAL;
  return Q4KV_OK;
}

// Every decode kernel keeps its partial records behind a header of fixed size (the arrival counters
// of the kernels that merge in the same launch), so that one workspace serves any sequence of calls.
size_t workspace_need(const Layout& y, int n_agents, int max_kv_len, int total_q) {
  if (total_q > 0) return 16;   // the prefill path keeps no partials
  const DecodePlan p = plan_decode(y, n_agents, max_kv_len, 0);
  size_t need = (size_t)n_agents * y.Hq * p.n_splits * (y.Dv + 2) * sizeof(float) + 16;
  if (decode_mla_supported(y)) {
    const size_t mla = decode_mla_workspace_bytes(y, n_agents, max_kv_len);
    if (mla > need) need = mla;
  }
  if (decode_mma_supported(y)) {
    const size_t mma = decode_mma_workspace_bytes(y, n_agents);
    if (mma > need) need = mma;
  }
  return kWorkspaceHeaderBytes + need;
}

// The kernels that expand the cache into binary16 tiles round each dequantized element once; they are taken only when
// the spec allows it and the softmax scale is at most 2 / sqrt(d_qk) (the error a rounded key leaves in a score grows
// with the scale).  Everything else multiplies the codes exactly.  Bfloat16 scales and biases are converted to binary16
// once per key block by those kernels (exact for every magnitude a cache written by this library can hold; a magnitude
// beyond binary16's largest number, which only a foreign cache can hold, raises Q4KV_FLAG_SB_RANGE).
bool tiles_allowed(const q4kv_spec* s, float softmax_scale) {
  return s->exact_products == 0 && softmax_scale > 0.f && softmax_scale * softmax_scale * (float)s->d_qk <= 4.f;
}

}  // namespace

extern "C" {

const char* q4kv_status_string(int code) {
  switch (code) {
    case Q4KV_OK: return "ok";
    case Q4KV_EINVAL: return "invalid argument (null, negative or misaligned)";
    case Q4KV_EUNSUPPORTED: return "spec not supported by this library";
    case Q4KV_EWORKSPACE: return "workspace or destination buffer too small";
    case Q4KV_ECUDA: return "CUDA launch or runtime error";
    default: return "unknown status";
  }
}

size_t q4kv_pool_bytes(const q4kv_spec* spec, int32_t n_blocks) {
  if (check_spec(spec) != Q4KV_OK || n_blocks <= 0) return 0;
  const Layout y = make_layout(*spec, n_blocks);
  return (size_t)y.L * y.layer_bytes;
}

size_t q4kv_packed_bytes(const q4kv_spec* spec, int32_t n_tokens) {
  if (check_spec(spec) != Q4KV_OK || n_tokens < 0) return 0;
  const Layout y = make_layout(*spec, 1);
  const uint64_t nblk = ((uint64_t)n_tokens + kBlockTokens - 1) / kBlockTokens;
  return (size_t)(y.L * nblk * persisted_block_bytes(y));
}

size_t q4kv_workspace_bytes(const q4kv_spec* spec, int32_t n_agents, int32_t max_kv_len, int32_t total_q) {
  if (check_spec(spec) != Q4KV_OK || n_agents < 0 || max_kv_len < 0 || total_q < 0) return 0;
  const Layout y = make_layout(*spec, 1);
  return workspace_need(y, n_agents > 0 ? n_agents : 1, max_kv_len > 0 ? max_kv_len : 1, total_q);
}

int q4kv_quantize_append(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer,
                         const q4kv_batch* batch, const int32_t* pos, const int32_t* new_offs,
                         int32_t total_new, const void* k_new, const void* v_new,
                         int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if ((rc = check_batch(batch))) return rc;
  if (!pool || n_blocks <= 0 || layer < 0 || layer >= spec->n_layers || total_new < 0) return Q4KV_EINVAL;
  if (total_new == 0 || batch->n_agents == 0) return Q4KV_OK;
  if (!pos || !new_offs || !k_new) return Q4KV_EINVAL;
  if ((spec->v_aliases_k != 0) != (v_new == nullptr)) return Q4KV_EINVAL;
  if (!aligned16(pool) || !aligned16(k_new) || !aligned16(v_new)) return Q4KV_EINVAL;
  const Layout y = make_layout(*spec, n_blocks);
  const cudaError_t e = launch_quantize_append(y, pool, n_blocks, layer, *batch, pos, new_offs, total_new, k_new,
                                               v_new, status_flags, (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_decode_attention(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                          const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                          int32_t window, const void* q, float softmax_scale,
                          void* out, int32_t out_dtype, float* lse,
                          void* workspace, size_t workspace_bytes,
                          int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if ((rc = check_batch(batch))) return rc;
  if (!pool || n_blocks <= 0 || layer < 0 || layer >= spec->n_layers || window < 0 || max_kv_len < 0) return Q4KV_EINVAL;
  if (out_dtype != Q4KV_OUT_F32 && out_dtype != Q4KV_OUT_BF16) return Q4KV_EINVAL;
  if (batch->n_agents == 0) return Q4KV_OK;
  if (!kv_lens || !q || !out || !workspace) return Q4KV_EINVAL;
  if (!aligned16(pool) || !aligned16(q) || !aligned16(out) || !aligned16(workspace)) return Q4KV_EINVAL;
  const int cap = batch->max_blocks * kBlockTokens;
  if (max_kv_len == 0 || max_kv_len > cap) max_kv_len = cap;
  const Layout y = make_layout(*spec, n_blocks);
  if (workspace_bytes < workspace_need(y, batch->n_agents, max_kv_len, 0)) return Q4KV_EWORKSPACE;
  void* records = (uint8_t*)workspace + kWorkspaceHeaderBytes;
  cudaError_t e;
  if (decode_mla_supported(y))
    e = launch_decode_mla(y, pool, n_blocks, layer, *batch, kv_lens, max_kv_len, window, q, softmax_scale, out, out_dtype,
                          lse, records, status_flags, (cudaStream_t)stream, nullptr, !tiles_allowed(spec, softmax_scale));
  else if (decode_mma_supported(y) && decode_mma_fits(y, batch->n_agents, batch->max_blocks))
    e = launch_decode_mma(y, pool, n_blocks, layer, *batch, kv_lens, max_kv_len, &window, 1, q, softmax_scale, out,
                          out_dtype, lse, workspace, status_flags, (cudaStream_t)stream);
  else
    e = launch_attention_generic(y, pool, n_blocks, layer, *batch, kv_lens, nullptr, 0, 1, max_kv_len, window, q,
                                 softmax_scale, out, out_dtype, lse, records, status_flags, (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_append_decode_attention(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer,
                                 const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 int32_t window, const void* k_new, const void* v_new,
                                 const void* q, float softmax_scale,
                                 void* out, int32_t out_dtype, float* lse,
                                 void* workspace, size_t workspace_bytes,
                                 int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if ((rc = check_batch(batch))) return rc;
  if (!pool || n_blocks <= 0 || layer < 0 || layer >= spec->n_layers || window < 0 || max_kv_len < 0) return Q4KV_EINVAL;
  if (out_dtype != Q4KV_OUT_F32 && out_dtype != Q4KV_OUT_BF16) return Q4KV_EINVAL;
  if (batch->n_agents == 0) return Q4KV_OK;
  const bool need_v = !spec->v_aliases_k;                  // an aliased cache stores no V rows
  if (!kv_lens || !q || !out || !workspace || !k_new || (need_v && !v_new)) return Q4KV_EINVAL;
  if (!aligned16(pool) || !aligned16(q) || !aligned16(out) || !aligned16(workspace) || !aligned16(k_new) ||
      (need_v && !aligned16(v_new)))
    return Q4KV_EINVAL;
  const int cap = batch->max_blocks * kBlockTokens;
  if (max_kv_len == 0 || max_kv_len > cap) max_kv_len = cap;
  const Layout y = make_layout(*spec, n_blocks);
  if (decode_mla_supported(y)) {
    if (workspace_bytes < workspace_need(y, batch->n_agents, max_kv_len, 0)) return Q4KV_EWORKSPACE;
    const cudaError_t e = launch_decode_mla(y, pool, n_blocks, layer, *batch, kv_lens, max_kv_len, window, q, softmax_scale,
                                            out, out_dtype, lse, (uint8_t*)workspace + kWorkspaceHeaderBytes, status_flags,
                                            (cudaStream_t)stream, k_new, !tiles_allowed(spec, softmax_scale));
    return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
  }
  if (!decode_mma_supported(y) || !decode_mma_fits(y, batch->n_agents, batch->max_blocks)) return Q4KV_EUNSUPPORTED;
  if (workspace_bytes < workspace_need(y, batch->n_agents, max_kv_len, 0)) return Q4KV_EWORKSPACE;
  const cudaError_t e = launch_decode_mma(y, pool, n_blocks, layer, *batch, kv_lens, max_kv_len, &window, 1, q, softmax_scale,
                                          out, out_dtype, lse, workspace, status_flags, (cudaStream_t)stream, k_new, v_new);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

size_t q4kv_workspace_bytes_layers(const q4kv_spec* spec, int32_t n_agents, int32_t max_kv_len, int32_t layer_count) {
  if (check_spec(spec) != Q4KV_OK || n_agents < 0 || max_kv_len < 0 || layer_count < 1) return 0;
  const Layout y = make_layout(*spec, 1);
  if (!decode_mma_supported(y)) return 0;
  const size_t one = workspace_need(y, n_agents > 0 ? n_agents : 1, max_kv_len > 0 ? max_kv_len : 1, 0);
  const size_t all = kWorkspaceHeaderBytes + decode_mma_workspace_bytes(y, n_agents > 0 ? n_agents : 1, layer_count);
  return all > one ? all : one;
}

int q4kv_decode_attention_layers(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer_begin,
                                 int32_t layer_count, const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 const int32_t* windows, const void* k_new, const void* v_new, const void* q,
                                 float softmax_scale, void* out, int32_t out_dtype, float* lse,
                                 void* workspace, size_t workspace_bytes, int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if ((rc = check_batch(batch))) return rc;
  if (!pool || n_blocks <= 0 || layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > spec->n_layers ||
      max_kv_len < 0 || !windows)
    return Q4KV_EINVAL;
  for (int i = 0; i < layer_count; ++i)
    if (windows[i] < 0) return Q4KV_EINVAL;
  if (out_dtype != Q4KV_OUT_F32 && out_dtype != Q4KV_OUT_BF16) return Q4KV_EINVAL;
  if (batch->n_agents == 0) return Q4KV_OK;
  if (!kv_lens || !q || !out || !workspace || ((k_new == nullptr) != (v_new == nullptr))) return Q4KV_EINVAL;
  if (!aligned16(pool) || !aligned16(q) || !aligned16(out) || !aligned16(workspace) || !aligned16(k_new) || !aligned16(v_new))
    return Q4KV_EINVAL;
  const int cap = batch->max_blocks * kBlockTokens;
  if (max_kv_len == 0 || max_kv_len > cap) max_kv_len = cap;
  const Layout y = make_layout(*spec, n_blocks);
  if (!decode_mma_supported(y) || !decode_mma_fits(y, batch->n_agents, batch->max_blocks, layer_count)) return Q4KV_EUNSUPPORTED;
  if (workspace_bytes < kWorkspaceHeaderBytes + decode_mma_workspace_bytes(y, batch->n_agents, layer_count)) return Q4KV_EWORKSPACE;
  const cudaError_t e = launch_decode_mma(y, pool, n_blocks, layer_begin, *batch, kv_lens, max_kv_len, windows, layer_count, q,
                                          softmax_scale, out, out_dtype, lse, workspace, status_flags, (cudaStream_t)stream,
                                          k_new, v_new);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_prefill_attention(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                           const q4kv_batch* batch, const int32_t* kv_lens, const int32_t* q_offs,
                           int32_t total_q, int32_t max_q_len, int32_t max_kv_len,
                           int32_t window, const void* q, float softmax_scale,
                           void* out, int32_t out_dtype, float* lse,
                           void* workspace, size_t workspace_bytes,
                           int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if ((rc = check_batch(batch))) return rc;
  if (!pool || n_blocks <= 0 || layer < 0 || layer >= spec->n_layers || window < 0 || max_kv_len < 0 ||
      total_q < 0 || max_q_len < 0)
    return Q4KV_EINVAL;
  if (out_dtype != Q4KV_OUT_F32 && out_dtype != Q4KV_OUT_BF16) return Q4KV_EINVAL;
  if (batch->n_agents == 0 || total_q == 0) return Q4KV_OK;
  if (!kv_lens || !q_offs || !q || !out || !workspace) return Q4KV_EINVAL;
  if (!aligned16(pool) || !aligned16(q) || !aligned16(out) || !aligned16(workspace)) return Q4KV_EINVAL;
  const int cap = batch->max_blocks * kBlockTokens;
  if (max_kv_len == 0 || max_kv_len > cap) max_kv_len = cap;
  if (max_q_len == 0 || max_q_len > total_q) max_q_len = total_q;
  const Layout y = make_layout(*spec, n_blocks);
  if (workspace_bytes < workspace_need(y, batch->n_agents, max_kv_len, total_q)) return Q4KV_EWORKSPACE;
  cudaError_t e;
  if (prefill_umma_supported(y) && tiles_allowed(spec, softmax_scale))
    e = launch_prefill_umma(y, pool, n_blocks, layer, *batch, kv_lens, q_offs, max_q_len, window, q, softmax_scale, out,
                            out_dtype, lse, status_flags, (cudaStream_t)stream);
  else if (prefill_umma_1tile_supported(y) && tiles_allowed(spec, softmax_scale))
    e = launch_prefill_umma_1tile(y, pool, n_blocks, layer, *batch, kv_lens, q_offs, max_q_len, window, q, softmax_scale,
                                  out, out_dtype, lse, status_flags, (cudaStream_t)stream);
  else if (prefill_mma_supported(y))
    e = launch_prefill_mma(y, pool, n_blocks, layer, *batch, kv_lens, q_offs, max_q_len, window, q, softmax_scale, out,
                           out_dtype, lse, status_flags, (cudaStream_t)stream);
  else
    e = launch_attention_generic(y, pool, n_blocks, layer, *batch, kv_lens, q_offs, total_q, max_q_len, max_kv_len,
                                 window, q, softmax_scale, out, out_dtype, lse, workspace, status_flags,
                                 (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_pack(const q4kv_spec* spec, const void* pool, int32_t n_blocks,
              const int32_t* block_table_row, int32_t n_tokens,
              void* dst, size_t dst_bytes, int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if (!pool || n_blocks <= 0 || n_tokens < 0) return Q4KV_EINVAL;
  if (n_tokens == 0) return Q4KV_OK;
  if (!block_table_row || !dst || !aligned16(pool) || !aligned16(dst)) return Q4KV_EINVAL;
  if (dst_bytes < q4kv_packed_bytes(spec, n_tokens)) return Q4KV_EWORKSPACE;
  const Layout y = make_layout(*spec, n_blocks);
  const cudaError_t e = launch_pack(y, pool, n_blocks, block_table_row, n_tokens, dst, status_flags, (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_unpack(const q4kv_spec* spec, const void* src, size_t src_bytes, int32_t n_tokens,
                void* pool, int32_t n_blocks, const int32_t* block_table_row,
                int32_t* status_flags, void* stream) {
  int rc = check_spec(spec);
  if (rc) return rc;
  if (!pool || n_blocks <= 0 || n_tokens < 0) return Q4KV_EINVAL;
  if (n_tokens == 0) return Q4KV_OK;
  if (!block_table_row || !src || !aligned16(pool) || !aligned16(src)) return Q4KV_EINVAL;
  if (src_bytes < q4kv_packed_bytes(spec, n_tokens)) return Q4KV_EWORKSPACE;
  const Layout y = make_layout(*spec, n_blocks);
  const cudaError_t e = launch_unpack(y, src, n_tokens, pool, n_blocks, block_table_row, status_flags, (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

}  // extern "C"
