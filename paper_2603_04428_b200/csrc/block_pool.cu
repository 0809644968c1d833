// Block pool bookkeeping and the dense-batch shim (Section 3.1 "Block Pool with Per-Agent Isolation"; Section 3.4
// BatchQuantizedKVCache.merge / extract).
//
// The allocator is host-side policy: it hands out the pool's 256-token blocks to agents (each block belongs to one agent
// at a time, so no agent can read another's cache), keeps a least-recently-used order of the agents, and names the
// agent to evict when the pool is full.  It never touches device memory; persisting a victim before its blocks are
// reused is the caller's step (q4kv_save), which is why eviction is a two-call affair: pick, then release.
//
// merge / extract exist in the paper because its framework attends over dense tensors: caches of different lengths
// are left-padded to a common length and stacked.  This library attends through block tables and needs neither, but
// code written against the dense form can move a layer's batch into the pool (merge) and out of it (extract).
#include <cstdlib>
#include <cstring>
#include <list>
#include <new>
#include <unordered_map>
#include <vector>

#include "q4kv_layout.cuh"

using namespace q4kv;

struct q4kv_allocator {
  struct Agent {
    std::vector<int32_t> blocks;
    bool pinned = false;
    std::list<int64_t>::iterator lru_pos;
  };
  int32_t n_blocks = 0;
  std::vector<int32_t> free_list;                    // a stack: the most recently freed block is reused first
  std::unordered_map<int64_t, Agent> agents;
  std::list<int64_t> lru;                            // front: least recently used
};

namespace {

void touch(q4kv_allocator* al, q4kv_allocator::Agent& ag, int64_t id) {
  al->lru.erase(ag.lru_pos);
  al->lru.push_back(id);
  ag.lru_pos = std::prev(al->lru.end());
}

size_t dense_need(const q4kv_spec* spec, int32_t n_agents, int32_t T) {
  const Layout y = make_layout(*spec, 1);
  const size_t rows = (size_t)n_agents * y.Hkv * T;
  return rows * ((size_t)y.D / 2 + 4 * y.G + (y.alias ? 0 : (size_t)y.Dv / 2 + 4 * y.Gv));
}

int dense_call(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer, const q4kv_batch* batch,
               const int32_t* kv_lens, int32_t T, void* dense, size_t dense_bytes, bool to_pool, int32_t* flags,
               void* stream) {
  if (!spec || !batch || !pool || n_blocks <= 0 || T <= 0 || batch->n_agents < 0 || batch->max_blocks <= 0) return Q4KV_EINVAL;
  if (q4kv_pool_bytes(spec, n_blocks) == 0) return Q4KV_EUNSUPPORTED;
  if (layer < 0 || layer >= spec->n_layers) return Q4KV_EINVAL;
  if (batch->n_agents == 0) return Q4KV_OK;
  if (!kv_lens || !dense || !batch->block_tables) return Q4KV_EINVAL;
  if ((reinterpret_cast<uintptr_t>(pool) | reinterpret_cast<uintptr_t>(dense)) & 15u) return Q4KV_EINVAL;
  const size_t need = dense_need(spec, batch->n_agents, T);
  if (dense_bytes < need) return Q4KV_EWORKSPACE;
  const Layout y = make_layout(*spec, n_blocks);
  cudaStream_t st = (cudaStream_t)stream;
  if (!to_pool && cudaMemsetAsync(dense, 0, need, st) != cudaSuccess) return Q4KV_ECUDA;   // the left padding is zero bytes
  const cudaError_t e = launch_dense_exchange(y, pool, n_blocks, layer, *batch, kv_lens, T, dense, to_pool, flags, st);
  return e == cudaSuccess ? Q4KV_OK : Q4KV_ECUDA;
}

}  // namespace

extern "C" {

q4kv_allocator* q4kv_allocator_create(int32_t n_blocks) {
  if (n_blocks <= 0) return nullptr;
  q4kv_allocator* al = new (std::nothrow) q4kv_allocator;
  if (!al) return nullptr;
  al->n_blocks = n_blocks;
  al->free_list.reserve(n_blocks);
  for (int32_t b = n_blocks - 1; b >= 0; --b) al->free_list.push_back(b);   // block 0 is handed out first
  return al;
}

void q4kv_allocator_destroy(q4kv_allocator* al) { delete al; }

int32_t q4kv_allocator_free_blocks(const q4kv_allocator* al) { return al ? (int32_t)al->free_list.size() : -1; }

int32_t q4kv_allocator_agent_blocks(const q4kv_allocator* al, int64_t agent_id) {
  if (!al) return -1;
  const auto it = al->agents.find(agent_id);
  return it == al->agents.end() ? 0 : (int32_t)it->second.blocks.size();
}

int q4kv_allocator_reserve(q4kv_allocator* al, int64_t agent_id, int32_t n_tokens, int32_t* table_row, int32_t max_blocks) {
  if (!al || n_tokens < 0 || !table_row || max_blocks <= 0) return Q4KV_EINVAL;
  const int32_t want = (n_tokens + kBlockTokens - 1) / kBlockTokens;
  if (want > max_blocks) return Q4KV_EINVAL;
  auto it = al->agents.find(agent_id);
  const int32_t have = it == al->agents.end() ? 0 : (int32_t)it->second.blocks.size();
  if (want > have && (size_t)(want - have) > al->free_list.size()) return Q4KV_EWORKSPACE;   // evict first (pick a victim)
  if (it == al->agents.end()) {
    it = al->agents.emplace(agent_id, q4kv_allocator::Agent()).first;
    al->lru.push_back(agent_id);
    it->second.lru_pos = std::prev(al->lru.end());
  } else {
    touch(al, it->second, agent_id);
  }
  q4kv_allocator::Agent& ag = it->second;
  while ((int32_t)ag.blocks.size() < want) { ag.blocks.push_back(al->free_list.back()); al->free_list.pop_back(); }
  for (int32_t i = 0; i < max_blocks; ++i) table_row[i] = i < (int32_t)ag.blocks.size() ? ag.blocks[i] : -1;
  return Q4KV_OK;
}

int q4kv_allocator_touch(q4kv_allocator* al, int64_t agent_id) {
  if (!al) return Q4KV_EINVAL;
  const auto it = al->agents.find(agent_id);
  if (it == al->agents.end()) return Q4KV_EINVAL;
  touch(al, it->second, agent_id);
  return Q4KV_OK;
}

int q4kv_allocator_pin(q4kv_allocator* al, int64_t agent_id, int32_t pinned) {
  if (!al) return Q4KV_EINVAL;
  const auto it = al->agents.find(agent_id);
  if (it == al->agents.end()) return Q4KV_EINVAL;
  it->second.pinned = pinned != 0;
  return Q4KV_OK;
}

int q4kv_allocator_pick_victim(const q4kv_allocator* al, int64_t* agent_id) {
  if (!al || !agent_id) return Q4KV_EINVAL;
  for (const int64_t id : al->lru) {
    const auto it = al->agents.find(id);
    if (it != al->agents.end() && !it->second.pinned && !it->second.blocks.empty()) { *agent_id = id; return Q4KV_OK; }
  }
  return Q4KV_EWORKSPACE;                              // every agent that holds blocks is pinned
}

int q4kv_allocator_release(q4kv_allocator* al, int64_t agent_id) {
  if (!al) return Q4KV_EINVAL;
  const auto it = al->agents.find(agent_id);
  if (it == al->agents.end()) return Q4KV_EINVAL;
  for (auto b = it->second.blocks.rbegin(); b != it->second.blocks.rend(); ++b) al->free_list.push_back(*b);
  al->lru.erase(it->second.lru_pos);
  al->agents.erase(it);
  return Q4KV_OK;
}

size_t q4kv_dense_bytes(const q4kv_spec* spec, int32_t n_agents, int32_t T) {
  if (!spec || n_agents < 0 || T < 0 || q4kv_pool_bytes(spec, 1) == 0) return 0;
  return dense_need(spec, n_agents, T);
}

int q4kv_merge_dense(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer, const q4kv_batch* batch,
                     const int32_t* kv_lens, int32_t T, const void* dense, size_t dense_bytes, int32_t* status_flags,
                     void* stream) {
  return dense_call(spec, pool, n_blocks, layer, batch, kv_lens, T, const_cast<void*>(dense), dense_bytes, true, status_flags,
                    stream);
}

int q4kv_extract_dense(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer, const q4kv_batch* batch,
                       const int32_t* kv_lens, int32_t T, void* dense, size_t dense_bytes, int32_t* status_flags,
                       void* stream) {
  return dense_call(spec, const_cast<void*>(pool), n_blocks, layer, batch, kv_lens, T, dense, dense_bytes, false, status_flags,
                    stream);
}

}  // extern "C"
