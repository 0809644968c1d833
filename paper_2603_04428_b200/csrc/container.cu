// The persisted container of one agent's cache and the warm-restore leg (Appendix "safetensors Q4 Format";
// Section 3.2 "Q4 Quantization Pipeline": the cache goes to disk in its quantized form and comes back without a
// dequantize/requantize step; the warm-cache rows of the time-to-first-token table).
//
// File = a safetensors file: 8 bytes (little-endian length N of the header), N bytes of JSON, then the data section,
// which is exactly the buffer q4kv_pack writes.  The header names every tensor of every layer and block,
// L{l}_B{b}_{K,V}_{weights,scales,biases}, with its dtype, shape and byte range in the data section, and carries the
// cache spec and the token count as metadata.  The header text is canonical (fixed key order, no blanks, padded with
// spaces to a multiple of 64 bytes), so the same cache always gives the same file.
//
// Restore = pinned host memory -> device staging -> q4kv_unpack, in chunks of whole layers: the copy of chunk c + 1
// runs on the copy stream while chunk c is scattered into the pool on the unpack stream (two staging halves, two
// events each).  One cudaMemcpyAsync per chunk.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>

#include "q4kv_layout.cuh"

using namespace q4kv;

namespace {

constexpr const char* kFormatTag = "q4kv-1";

void put_tensor(std::string& js, int l, int b, const char* kv, const char* what, const char* dtype, int h, int d2,
                uint64_t& off, uint64_t bytes) {
  char buf[256];
  std::snprintf(buf, sizeof buf, ",\"L%d_B%d_%s_%s\":{\"dtype\":\"%s\",\"shape\":[%d,256,%d],\"data_offsets\":[%llu,%llu]}", l, b,
                kv, what, dtype, h, d2, (unsigned long long)off, (unsigned long long)(off + bytes));
  js += buf;
  off += bytes;
}

// canonical header text (without the length prefix and the padding)
std::string header_json(const q4kv_spec& s, int n_tokens) {
  const Layout y = make_layout(s, 1);
  const int nblk = (n_tokens + kBlockTokens - 1) / kBlockTokens;
  char buf[512];
  std::snprintf(buf, sizeof buf,
                "{\"__metadata__\":{\"format\":\"%s\",\"n_layers\":\"%d\",\"n_q_heads\":\"%d\",\"n_kv_heads\":\"%d\",\"d_qk\":\"%d\","
                "\"d_v\":\"%d\",\"v_aliases_k\":\"%d\",\"group\":\"%d\",\"block_tokens\":\"%d\",\"sb_dtype\":\"%d\",\"n_tokens\":\"%d\"}",
                kFormatTag, s.n_layers, s.n_q_heads, s.n_kv_heads, s.d_qk, s.d_v, s.v_aliases_k ? 1 : 0, s.group,
                s.block_tokens, s.sb_dtype, n_tokens);
  std::string js = buf;
  js.reserve(js.size() + (size_t)s.n_layers * nblk * 6 * 100);
  const char* sbt = s.sb_dtype == 1 ? "BF16" : "F16";
  uint64_t off = 0;
  const uint64_t rows = (uint64_t)y.Hkv * kBlockTokens;
  for (int l = 0; l < s.n_layers; ++l)
    for (int b = 0; b < nblk; ++b) {
      put_tensor(js, l, b, "K", "weights", "U32", y.Hkv, y.D / 8, off, rows * (y.D / 8) * 4);
      put_tensor(js, l, b, "K", "scales", sbt, y.Hkv, y.G, off, rows * y.G * 2);
      put_tensor(js, l, b, "K", "biases", sbt, y.Hkv, y.G, off, rows * y.G * 2);
      if (!y.alias) {
        put_tensor(js, l, b, "V", "weights", "U32", y.Hkv, y.Dv / 8, off, rows * (y.Dv / 8) * 4);
        put_tensor(js, l, b, "V", "scales", sbt, y.Hkv, y.Gv, off, rows * y.Gv * 2);
        put_tensor(js, l, b, "V", "biases", sbt, y.Hkv, y.Gv, off, rows * y.Gv * 2);
      }
    }
  js += "}";
  return js;
}

size_t padded_header_bytes(size_t json_bytes) { return (8 + json_bytes + 63) & ~(size_t)63; }

bool spec_ok(const q4kv_spec* s) {
  return s && s->n_layers > 0 && s->n_q_heads > 0 && s->n_kv_heads > 0 && s->d_qk > 0 && s->d_v > 0 && s->group == 64 &&
         s->block_tokens == 256 && (s->sb_dtype == 0 || s->sb_dtype == 1) && s->d_qk % 64 == 0 && s->d_v % 64 == 0 &&
         s->n_q_heads % s->n_kv_heads == 0 && s->d_qk <= 1024 && s->d_v <= 512 && (!s->v_aliases_k || s->d_v <= s->d_qk);
}

// value of "key":"<digits>" inside the metadata object; false when absent or malformed
bool meta_int(const std::string& js, const char* key, int* out) {
  const std::string pat = std::string("\"") + key + "\":\"";
  const size_t at = js.find(pat);
  if (at == std::string::npos) return false;
  size_t i = at + pat.size();
  long v = 0;
  int digits = 0;
  while (i < js.size() && js[i] >= '0' && js[i] <= '9' && digits < 10) { v = v * 10 + (js[i] - '0'); ++i; ++digits; }
  if (digits == 0 || i >= js.size() || js[i] != '"' || v > 0x7fffffffL) return false;
  *out = (int)v;
  return true;
}

}  // namespace

extern "C" {

size_t q4kv_container_header_bytes(const q4kv_spec* spec, int32_t n_tokens) {
  if (!spec_ok(spec) || n_tokens < 0) return 0;
  return padded_header_bytes(header_json(*spec, n_tokens).size());
}

int q4kv_container_write_header(const q4kv_spec* spec, int32_t n_tokens, void* dst, size_t dst_bytes) {
  if (!spec || !dst || n_tokens < 0) return Q4KV_EINVAL;
  if (!spec_ok(spec)) return Q4KV_EUNSUPPORTED;
  const std::string js = header_json(*spec, n_tokens);
  const size_t total = padded_header_bytes(js.size());
  if (dst_bytes < total) return Q4KV_EWORKSPACE;
  const uint64_t n = total - 8;
  uint8_t* d = (uint8_t*)dst;
  for (int i = 0; i < 8; ++i) d[i] = (uint8_t)(n >> (8 * i));
  std::memcpy(d + 8, js.data(), js.size());
  std::memset(d + 8 + js.size(), ' ', total - 8 - js.size());
  return Q4KV_OK;
}

int q4kv_container_read_header(const void* src, size_t src_bytes, q4kv_spec* spec, int32_t* n_tokens, size_t* data_offset) {
  if (!src || !spec || !n_tokens || !data_offset || src_bytes < 8) return Q4KV_EINVAL;
  const uint8_t* s = (const uint8_t*)src;
  uint64_t n = 0;
  for (int i = 0; i < 8; ++i) n |= (uint64_t)s[i] << (8 * i);
  if (n < 2 || n > src_bytes - 8) return Q4KV_EINVAL;
  const std::string js((const char*)s + 8, (size_t)n);
  const size_t m0 = js.find("\"__metadata__\":{");
  if (m0 == std::string::npos) return Q4KV_EINVAL;
  const size_t m1 = js.find('}', m0);
  if (m1 == std::string::npos) return Q4KV_EINVAL;
  const std::string meta = js.substr(m0, m1 - m0 + 1);
  if (meta.find(std::string("\"format\":\"") + kFormatTag + "\"") == std::string::npos) return Q4KV_EUNSUPPORTED;
  q4kv_spec t;
  std::memset(&t, 0, sizeof t);
  int nt = 0;
  if (!meta_int(meta, "n_layers", &t.n_layers) || !meta_int(meta, "n_q_heads", &t.n_q_heads) ||
      !meta_int(meta, "n_kv_heads", &t.n_kv_heads) || !meta_int(meta, "d_qk", &t.d_qk) || !meta_int(meta, "d_v", &t.d_v) ||
      !meta_int(meta, "v_aliases_k", &t.v_aliases_k) || !meta_int(meta, "group", &t.group) ||
      !meta_int(meta, "block_tokens", &t.block_tokens) || !meta_int(meta, "sb_dtype", &t.sb_dtype) ||
      !meta_int(meta, "n_tokens", &nt))
    return Q4KV_EINVAL;
  if (!spec_ok(&t)) return Q4KV_EUNSUPPORTED;
  // the tensor table must be the canonical one for this spec and token count: then every byte range is known
  const std::string want = header_json(t, nt);
  if (js.compare(0, want.size(), want) != 0) return Q4KV_EINVAL;
  for (size_t i = want.size(); i < js.size(); ++i)
    if (js[i] != ' ') return Q4KV_EINVAL;
  if (src_bytes - 8 - n < q4kv_packed_bytes(&t, nt) && src_bytes != 8 + n) return Q4KV_EINVAL;   // a truncated data section
  *spec = t;
  *n_tokens = nt;
  *data_offset = 8 + (size_t)n;
  return Q4KV_OK;
}

int q4kv_save(const q4kv_spec* spec, const void* pool, int32_t n_blocks, const int32_t* block_table_row, int32_t n_tokens,
              void* dev_staging, size_t dev_staging_bytes, void* host_image, size_t host_image_bytes,
              int32_t* status_flags, void* stream) {
  if (!spec || !pool || !block_table_row || !dev_staging || !host_image || n_tokens <= 0) return Q4KV_EINVAL;
  const size_t hb = q4kv_container_header_bytes(spec, n_tokens);
  const size_t pb = q4kv_packed_bytes(spec, n_tokens);
  if (hb == 0 || pb == 0) return Q4KV_EUNSUPPORTED;
  if (dev_staging_bytes < pb || host_image_bytes < hb + pb) return Q4KV_EWORKSPACE;
  int rc = q4kv_container_write_header(spec, n_tokens, host_image, hb);
  if (rc != Q4KV_OK) return rc;
  rc = q4kv_pack(spec, pool, n_blocks, block_table_row, n_tokens, dev_staging, dev_staging_bytes, status_flags, stream);
  if (rc != Q4KV_OK) return rc;
  const cudaError_t e = cudaMemcpyAsync((uint8_t*)host_image + hb, dev_staging, pb, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

int q4kv_restore(const q4kv_spec* spec, const void* host_packed, size_t packed_bytes, int32_t n_tokens, void* pool,
                 int32_t n_blocks, const int32_t* block_table_row, void* dev_staging, size_t dev_staging_bytes,
                 int32_t* status_flags, void* copy_stream, void* unpack_stream) {
  if (!spec || !host_packed || !pool || !block_table_row || !dev_staging || n_tokens <= 0 || n_blocks <= 0) return Q4KV_EINVAL;
  if (!spec_ok(spec)) return Q4KV_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(pool) | reinterpret_cast<uintptr_t>(dev_staging) | reinterpret_cast<uintptr_t>(host_packed)) & 15u)
    return Q4KV_EINVAL;
  const size_t pb = q4kv_packed_bytes(spec, n_tokens);
  if (packed_bytes < pb) return Q4KV_EWORKSPACE;
  const Layout y = make_layout(*spec, n_blocks);
  const size_t layer_bytes = pb / (size_t)y.L;
  // chunks of whole layers, two staging halves when they fit (else one: copy and scatter then alternate)
  const int halves = dev_staging_bytes >= 2 * layer_bytes ? 2 : 1;
  if (dev_staging_bytes < layer_bytes) return Q4KV_EWORKSPACE;
  const size_t half_bytes = (dev_staging_bytes / halves) & ~(size_t)255;
  int per_chunk = (int)(half_bytes / layer_bytes);
  if (per_chunk > y.L) per_chunk = y.L;
  // eight chunks at least when the cache has that many layers, so that most of the scatter hides behind the copies
  if (per_chunk > (y.L + 7) / 8) per_chunk = (y.L + 7) / 8;
  if (per_chunk < 1) per_chunk = 1;
  cudaStream_t cs = (cudaStream_t)copy_stream, us = (cudaStream_t)unpack_stream;
  cudaEvent_t copied[2] = {nullptr, nullptr}, freed[2] = {nullptr, nullptr};
  bool ok = true;
  for (int i = 0; i < halves && ok; ++i)
    ok = cudaEventCreateWithFlags(&copied[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&freed[i], cudaEventDisableTiming) == cudaSuccess;
  int rc = ok ? Q4KV_OK : Q4KV_ECUDA;
  int chunk = 0;
  for (int l0 = 0; l0 < y.L && rc == Q4KV_OK; l0 += per_chunk, ++chunk) {
    const int cnt = l0 + per_chunk <= y.L ? per_chunk : y.L - l0;
    const int h = chunk % halves;
    uint8_t* stage = (uint8_t*)dev_staging + (size_t)h * half_bytes;
    if (chunk >= halves && cudaStreamWaitEvent(cs, freed[h], 0) != cudaSuccess) { rc = Q4KV_ECUDA; break; }
    if (cudaMemcpyAsync(stage, (const uint8_t*)host_packed + (size_t)l0 * layer_bytes, (size_t)cnt * layer_bytes,
                        cudaMemcpyHostToDevice, cs) != cudaSuccess ||
        cudaEventRecord(copied[h], cs) != cudaSuccess || cudaStreamWaitEvent(us, copied[h], 0) != cudaSuccess) {
      rc = Q4KV_ECUDA;
      break;
    }
    if (launch_unpack_layers(y, stage, n_tokens, pool, n_blocks, block_table_row, status_flags, us, l0, cnt) != cudaSuccess ||
        cudaEventRecord(freed[h], us) != cudaSuccess) {
      rc = Q4KV_ECUDA;
      break;
    }
  }
  for (int i = 0; i < 2; ++i) {
    if (copied[i]) cudaEventDestroy(copied[i]);       // destruction is deferred until the recorded work has completed
    if (freed[i]) cudaEventDestroy(freed[i]);
  }
  return rc;
}

}  // extern "C"
