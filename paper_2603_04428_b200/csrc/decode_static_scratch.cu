// q4kv_decode_attention_static: decode attention for callers that cannot allocate device memory.
//
// Some hosts of this library have no allocator to offer at call time: an inference runtime that
// sized and handed out all of its device memory at start-up, a plugin loaded into a process whose
// memory pool it must not touch, code running between the capture-safe sections of a larger
// program.  They can pass the cache, the queries and the output, but not the scratch buffer that
// q4kv_decode_attention wants for its split partials.  This entry point supplies that scratch
// from a fixed array that lives in the library's own device image: loading the library reserves
// kStaticScratchBytes on every GPU that runs it, until the process exits, and nothing is
// allocated or freed by any call.
#include <mutex>

#include "q4kv_layout.cuh"

namespace {

constexpr size_t kStaticScratchBytes = Q4KV_STATIC_SCRATCH_BYTES;   // 8 MiB per device
constexpr int kMaxDevices = 64;

// In device code this names the array itself.  In host code the same name is only a handle for
// the runtime's symbol table, never an address a kernel may be given: the device address is
// asked for once per device with cudaGetSymbolAddress, while that device is current.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (set-up on first use per device).
int static_scratch(void** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return Q4KV_ECUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return Q4KV_ECUDA;
    g_scratch_ptr[dev] = p;
  }
  *ptr = g_scratch_ptr[dev];
  return Q4KV_OK;
}

}  // namespace

extern "C" {

int q4kv_decode_attention_static(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                                 const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 int32_t window, const void* q, float softmax_scale,
                                 void* out, int32_t out_dtype, float* lse,
                                 int32_t* status_flags, void* stream) {
  if (!spec || !batch) return Q4KV_EINVAL;
  // Reject what does not fit before touching the device: the array cannot grow.
  const int32_t cap = batch->max_blocks > 0 ? batch->max_blocks * q4kv::kBlockTokens : 0;
  const int32_t bound = (max_kv_len <= 0 || max_kv_len > cap) ? cap : max_kv_len;
  const size_t need = q4kv_workspace_bytes(spec, batch->n_agents, bound, 0);
  if (need == 0) return Q4KV_EUNSUPPORTED;
  if (need > kStaticScratchBytes) return Q4KV_EWORKSPACE;
  void* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != Q4KV_OK) return rc;
  // The arrival counters at the head of the scratch must be zero when the kernel starts.  A call that ran to its end
  // leaves them at zero, but one that gave up (Q4KV_FLAG_INTERNAL) may not have, and this caller has no buffer of its
  // own to clear: so every call clears the header first, with a memset enqueued on its stream (no allocation).  The
  // partial records behind the header are written before they are read within a call.
  if (cudaMemsetAsync(scratch, 0, q4kv::kWorkspaceHeaderBytes, (cudaStream_t)stream) != cudaSuccess) return Q4KV_ECUDA;
  return q4kv_decode_attention(spec, pool, n_blocks, layer, batch, kv_lens, max_kv_len, window, q, softmax_scale,
                               out, out_dtype, lse, scratch, kStaticScratchBytes, status_flags, stream);
}

}  // extern "C"
