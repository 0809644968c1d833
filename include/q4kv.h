/*
 * q4kv -- batched attention over 4-bit group-quantized KV caches, read in place.
 *
 * C ABI of the sm_100a library (libq4kv.so).  The operations are the hot path
 * behind the paper's BatchQuantizedKVCache (Section 3.4 "Batched Quantized
 * Inference"): quantize-and-append new K/V rows, attention of one query token
 * per agent over the whole Q4 cache, chunked-prefill attention of a new phase
 * over a cached Q4 prefix (Sections 3.4, 3.5), and the contiguous per-agent
 * layout that is persisted and restored (Appendix A).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers unless a comment says "host".  The
 *     spec and batch structs themselves are read on the HOST at call time.
 *   - The library owns no memory on this path: pool, block tables, lengths,
 *     q/out, workspace and the status word are caller-allocated device memory
 *     and must stay alive until the stream has run the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls are asynchronous: they validate on the host, enqueue kernels and
 *     return.  Nothing synchronises the device.
 *   - Return value: Q4KV_OK (0) or a negative Q4KV_E* code.  On a negative
 *     return nothing was launched.
 *   - Anomalies only visible on the device (a block id outside [0, n_blocks),
 *     a length beyond max_blocks*256, a negative length) OR the matching
 *     Q4KV_FLAG_* bit into *status_flags (int32, may be NULL), write zeros for
 *     the affected agent and carry on.  Kernels never trap, assert or wait.
 *   - Data pointers must be 16-byte aligned.
 *   - Calls on different streams are safe together when their outputs and
 *     workspaces do not overlap and none writes pool blocks another reads.
 *   - The kernels are launched with programmatic stream serialization: a
 *     kernel's prologue overlaps the tail of the preceding kernel of the
 *     stream, and it reads the lengths (kv_lens, pos, offsets) and block tables
 *     there.  The pool, q, new rows, outputs and workspace are touched only
 *     after the preceding kernels have completed.  Lengths and block tables
 *     must therefore not be written by a preceding kernel that itself signals
 *     its dependents early; an ordinary kernel, a copy or a memset is fine.
 *   - The library reads no environment variable; every choice is an argument.
 *
 * Q4 format (Section 3.2): groups of 64 consecutive head-dim elements; per
 * group one 16-bit scale and one 16-bit bias, both binary16 (sb_dtype 0) or
 * both bfloat16 (sb_dtype 1; Section 3.2 and Appendix A name both types);
 * 4-bit codes, value = code*scale + bias.  The quantizer's arithmetic is fixed
 * (single binary32 operations in this order) so that results are reproducible
 * bit for bit; the two roundings to 16 bits are taken in the cache's type:
 *     bias  = round_toward_minus_inf_16(min x)       (a zero is stored as +0)
 *     scale = round_toward_plus_inf_16( f32( f32(max x - bias) / 15 ) )
 *     code  = clamp( round_half_even( f32( f32(x - bias) / scale ) ), 0, 15 ),
 *             all codes 0 when scale == 0.
 * Inputs must be finite with |x| <= 65504.
 *
 * Block pool (Section 3.1): `pool` holds n_layers * n_blocks blocks of 256
 * tokens (all KV heads of one layer).  The byte layout inside the pool is
 * private to the library (it is arranged for the kernels' loads); exchange
 * cache contents through q4kv_pack / q4kv_unpack only.  A block table row lists,
 * for one agent, the physical block id of logical block 0, 1, ... ; the same
 * ids are used in every layer.
 */
#ifndef Q4KV_H
#define Q4KV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* The paper's ModelCacheSpec (Sections 3.1, 3.6): what a model's cache looks like. */
typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;
  int32_t n_kv_heads;    /* n_q_heads % n_kv_heads == 0; query head h reads KV head h / (n_q/n_kv) */
  int32_t d_qk;          /* key/query head dim, multiple of 64 (128, 256, 576, 192 ...)             */
  int32_t d_v;           /* value head dim, multiple of 64 (the paper's v_head_dim)                 */
  int32_t v_aliases_k;   /* 1: no V storage; the value row is the first d_v dims of the key row
                            (shared latent of MLA in absorbed form); requires d_v <= d_qk           */
  int32_t group;         /* quantization group, must be 64                                          */
  int32_t block_tokens;  /* tokens per pool block, must be 256                                      */
  int32_t sb_dtype;      /* scale/bias type: 0 = binary16, 1 = bfloat16.  Both take the same kernels; those
                            that work in binary16 convert a bfloat16 scale or bias first (see "Accuracy"
                            and Q4KV_FLAG_SB_RANGE)                                                  */
  int32_t exact_products;/* 0: attention kernels may expand the cache into binary16 tiles (one rounding
                            of every dequantized value, see "Accuracy" below); 1: always multiply the
                            4-bit codes exactly.  Ignored by append, pack and unpack.               */
} q4kv_spec;

/* One batch of agents. */
typedef struct {
  int32_t n_agents;
  int32_t max_blocks;            /* row length of block_tables                                      */
  const int32_t* block_tables;   /* device, [n_agents][max_blocks], physical ids in [0, n_blocks);
                                    entries past an agent's last block are never read              */
} q4kv_batch;

enum {
  Q4KV_OK = 0,
  Q4KV_EINVAL = -1,        /* null / negative / misaligned argument                                 */
  Q4KV_EUNSUPPORTED = -2,  /* spec outside what the kernels cover                                   */
  Q4KV_EWORKSPACE = -3,    /* workspace or destination buffer too small                             */
  Q4KV_ECUDA = -4          /* a CUDA launch or runtime call failed                                  */
};
enum {
  Q4KV_FLAG_BAD_BLOCK = 1,   /* a block id outside [0, n_blocks)                                    */
  Q4KV_FLAG_BAD_LENGTH = 2,  /* a length or position negative or beyond max_blocks*256              */
  Q4KV_FLAG_INTERNAL = 4,    /* a bounded wait inside a kernel ran out (the output is not valid)    */
  Q4KV_FLAG_SB_RANGE = 8     /* a bfloat16 scale or bias beyond binary16's largest number met a kernel that
                                expands the cache into binary16 tiles: the call's output is not valid
                                (such a cache lies outside what the tensor-core kernels carry, see
                                "Accuracy"; this library's quantizer never writes one)               */
};
enum { Q4KV_OUT_F32 = 0, Q4KV_OUT_BF16 = 1 };

/* Accuracy of the attention entry points (float32 output, against the attention over the exactly
 * dequantized values evaluated in float64).  Let M be the largest |code*scale + bias| among the
 * attended keys and values.
 *   - Kernels that multiply the 4-bit codes (decode with d_qk = d_v in {128, 256} or d_qk 192 / d_v 128
 *     and at most four query heads per KV head; decode on the MLA-latent cache when the tile kernel
 *     below is not allowed; prefill with d in {128, 256} when it is not; the shape-agnostic kernels
 *     every other case falls back to): the products are exact, sums are float32, the
 *     probabilities enter the value product as a two-term binary16 pair or as float32.  Error
 *     at most 2e-5 * M + 1e-5, i.e. within 2e-3 for any cache with M <= 64.  (An absolute bound:
 *     the tensor-core kernels carry probability x scale in binary16, so contributions of groups
 *     whose scale is below 2^-24 vanish; only bfloat16 caches can hold such scales.)
 *   - Kernels that expand the cache into binary16 tiles (prefill with d_qk = d_v in {128, 256} or d_qk 192 / d_v 128 and 1, 2 or 4
 *     query heads per KV head; decode on the MLA-latent cache: V aliasing K, d_qk 576, d_v 512, one
 *     KV head, at most 16 query heads) round every dequantized value once to binary16, a relative
 *     error of 2^-11 at most, and the probabilities likewise.  They are chosen only when
 *     exact_products == 0 and softmax_scale <= 2/sqrt(d_qk).  Their error is at most
 *     2^-10 * M * (1 + softmax_scale * ||q||_1 * M): the value and probability roundings, plus what
 *     the rounded keys do to the softmax weights.  A bfloat16 scale or bias enters as the binary16
 *     number of the same value: exact for magnitudes in [2^-14, 65504] (a bfloat16 number has 8
 *     significant bits), off by at most 2^-25 below that, so for bfloat16 caches add 2^-20 to the
 *     bound; a magnitude above 65504 raises Q4KV_FLAG_SB_RANGE.  The quantizer of this library never
 *     writes such a value (its inputs are bf16 numbers of magnitude at most 65504: the bias is then
 *     the group's minimum itself and the scale at most 8734); a cache persisted elsewhere should keep
 *     |code * scale + bias| <= 65504 as well: no tensor-core kernel here, exact or not, carries
 *     probability x scale beyond binary16's range.  On caches of unit-variance values (M about 5) the
 *     roundings average out over the attended keys and the measured error is below 3e-4; a cache
 *     with outlier channels or a gain (M >= 8) needs exact_products = 1 to stay within 2e-3. */

const char* q4kv_status_string(int code);

/* Sizes (host arithmetic only).  pool: n_layers*n_blocks blocks.  packed: whole blocks,
 * n_layers * ceil(n_tokens/256) * block bytes, block bytes = 256 * n_kv_heads *
 * (d_qk/2 + d_qk/16 [+ d_v/2 + d_v/16]) -- the h*d*n*(1+8/g) of Section 3.2.
 * workspace: scratch for split partials of q4kv_decode_attention (total_q = 0) or
 * q4kv_prefill_attention (total_q = number of query rows); max_kv_len bounds every length.
 * A zero return means the spec is not supported. */
size_t q4kv_pool_bytes(const q4kv_spec* spec, int32_t n_blocks);
size_t q4kv_packed_bytes(const q4kv_spec* spec, int32_t n_tokens);
size_t q4kv_workspace_bytes(const q4kv_spec* spec, int32_t n_agents, int32_t max_kv_len, int32_t total_q);

/* Quantize new K/V rows and write them into the agents' blocks -- the "update" half of
 * update-and-fetch (Section 3.4; format Section 3.2).
 *   pos      [A]   first cache position written for each agent (its current length)
 *   new_offs [A+1] prefix sums: agent a's new tokens are rows new_offs[a] .. new_offs[a+1]-1
 *   total_new      host copy of new_offs[A] (sizes the grid)
 *   k_new    bf16 [total_new][n_kv_heads][d_qk]
 *   v_new    bf16 [total_new][n_kv_heads][d_v]; must be NULL iff spec->v_aliases_k
 * Lengths are the caller's: this call does not bump them (the same lengths serve all layers).
 * Two agents must not share a block that either one writes. */
int q4kv_quantize_append(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer,
                         const q4kv_batch* batch, const int32_t* pos, const int32_t* new_offs,
                         int32_t total_new, const void* k_new, const void* v_new,
                         int32_t* status_flags, void* stream);

/* Decode attention: one query token per agent over that agent's whole Q4 cache, batched over
 * agents with ragged lengths (Sections 3.4, 3.6).  out = softmax(softmax_scale * q.K^T) . V over
 * the dequantized values, keys [lo, kv_len) with lo = max(0, kv_len - window) when window > 0
 * (sliding-window layers), lo = 0 when window == 0.
 *   kv_lens    [A]  cached tokens to attend (the query sits at position kv_len-1)
 *   max_kv_len      host upper bound on every kv_len (sizes the split grid); 0 = max_blocks*256.
 *                   An agent whose kv_len exceeds it is treated like any other bad length:
 *                   Q4KV_FLAG_BAD_LENGTH, zeros for that agent.
 *   q          bf16 [A][n_q_heads][d_qk]
 *   out        [A][n_q_heads][d_v], float32 or bf16 per out_dtype
 *   lse        optional float32 [A][n_q_heads], natural-log sum of exponentials; may be NULL
 *   workspace  at least q4kv_workspace_bytes(spec, A, max_kv_len, 0) bytes.  Its first
 *              Q4KV_WORKSPACE_HEADER_BYTES hold the arrival counters of the split merge: fill them
 *              with zero bytes once after allocating the workspace; every call finds them at zero
 *              and leaves them at zero, whatever the spec, the batch size or the kernel chosen, so
 *              one workspace sized for the largest batch serves all calls.  (If a call ever reports
 *              Q4KV_FLAG_INTERNAL, zero the header again.)  Nothing behind the header carries over
 *              between calls.
 * kv_len == 0 gives zeros and lse = -inf without a flag. */
#define Q4KV_WORKSPACE_HEADER_BYTES 65536u
int q4kv_decode_attention(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                          const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                          int32_t window, const void* q, float softmax_scale,
                          void* out, int32_t out_dtype, float* lse,
                          void* workspace, size_t workspace_bytes,
                          int32_t* status_flags, void* stream);

/* Update-and-fetch for one new token per agent in a single launch (Section 3.4: the cache's
 * update_and_fetch -- quantize the step's new K/V rows into the cache, then attend over it).
 * Equivalent to q4kv_quantize_append(pos = kv_lens - 1, one row per agent) followed by
 * q4kv_decode_attention(kv_lens): the pool ends up with the same bytes and the output is the same
 * attention, but the new token is quantized by the warp that attends its 32-token chunk, so no
 * second kernel runs.
 *   kv_lens  [A]  lengths INCLUDING the new token (it sits at position kv_len - 1); kv_len == 0:
 *                 nothing is appended for that agent
 *   k_new    bf16 [A][n_kv_heads][d_qk], v_new bf16 [A][n_kv_heads][d_v]: row a is agent a's token
 *                 (v_new is ignored, and may be NULL, when V aliases K)
 * All other arguments as in q4kv_decode_attention.  Covered specs: d_qk = d_v in {128, 256}, or d_qk 192
 * with d_v 128 (the per-head MLA cache of Section 3.6), with at most four query heads per KV head and V
 * not aliasing K; and the MLA-latent cache (V aliasing K, d_qk 576, d_v 512, one KV head, at most
 * 16 query heads), on the kernel q4kv_decode_attention would take for the same spec and scale.
 * Anything else returns Q4KV_EUNSUPPORTED and the caller makes the two calls.  Two agents must
 * not share the block that is written. */
int q4kv_append_decode_attention(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer,
                                 const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 int32_t window, const void* k_new, const void* v_new,
                                 const void* q, float softmax_scale,
                                 void* out, int32_t out_dtype, float* lse,
                                 void* workspace, size_t workspace_bytes,
                                 int32_t* status_flags, void* stream);

/* Update-and-fetch (or plain decode attention) for SEVERAL layers in one launch (Section 3.4; the same update_and_fetch,
 * batched over layers as well as agents).  For callers that hold the queries -- and, for the update, the new K/V rows --
 * of layers layer_begin .. layer_begin + layer_count - 1 at once (a replayed step, a speculative pass, a test harness):
 * the kernel's work list then runs over layers x agents x KV heads, so that small batches still fill the GPU.  Equivalent
 * to layer_count calls of q4kv_append_decode_attention (k_new, v_new given) or q4kv_decode_attention (both NULL), layer by
 * layer.
 *   windows  HOST [layer_count]: the sliding window of each layer (0: none)
 *   k_new    bf16 [layer_count][A][n_kv_heads][d_qk], v_new likewise with d_v; both NULL: nothing is appended
 *   q        bf16 [layer_count][A][n_q_heads][d_qk];  out [layer_count][A][n_q_heads][d_v];  lse [layer_count][A][n_q_heads]
 *   workspace  at least q4kv_workspace_bytes_layers(spec, A, max_kv_len, layer_count) bytes, header zeroed as for
 *              q4kv_decode_attention
 * Covered specs: d_qk = d_v in {128, 256}, at most four query heads per KV head, V not aliasing K, at most 64 layers
 * per call; anything else returns Q4KV_EUNSUPPORTED (call layer by layer then). */
size_t q4kv_workspace_bytes_layers(const q4kv_spec* spec, int32_t n_agents, int32_t max_kv_len, int32_t layer_count);
int q4kv_decode_attention_layers(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer_begin,
                                 int32_t layer_count, const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 const int32_t* windows, const void* k_new, const void* v_new, const void* q,
                                 float softmax_scale, void* out, int32_t out_dtype, float* lse,
                                 void* workspace, size_t workspace_bytes, int32_t* status_flags, void* stream);

/* Decode attention without a caller-supplied workspace.  The paper has no counterpart: this entry
 * point exists for hosts that cannot allocate device memory when they call -- a runtime that
 * carved up all of its device memory at start-up, a plugin that must not touch its host's
 * memory pool, code that runs where allocation calls are not allowed.  It computes exactly what
 * q4kv_decode_attention computes (same arguments, minus workspace and workspace_bytes), with the
 * split partials kept in a fixed array inside the library's device image instead.
 *   - The array is Q4KV_STATIC_SCRATCH_BYTES long.  Every GPU on which the library is loaded
 *     holds that much memory until the process exits, whether or not this entry point is used.
 *   - A batch whose q4kv_workspace_bytes(spec, n_agents, max_kv_len, 0) exceeds the array is
 *     rejected with Q4KV_EWORKSPACE and nothing is launched; use q4kv_decode_attention then.
 *   - No call allocates or frees anything (no cudaMalloc, no cudaFree, no library that would).
 *     The first call on each device looks up the array's device address (a host-side query, no
 *     launch); make that first call before any stream capture begins on that device.
 *   - All calls on one device share the one array, and it keeps whatever the last call left in
 *     it.  Each call first clears the arrival counters at the head of the array with a memset
 *     enqueued on its own stream (no allocation), so a call never depends on what an earlier one
 *     left there -- not even one that ended with Q4KV_FLAG_INTERNAL; the partial records behind
 *     the counters are written before they are read within a call.  Two calls that overlap on the
 *     GPU -- different streams, or one stream per thread -- race on the array and give wrong
 *     results: order them on one stream, or give the concurrent ones their own workspace through
 *     q4kv_decode_attention. */
#define Q4KV_STATIC_SCRATCH_BYTES (8u << 20)
int q4kv_decode_attention_static(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                                 const q4kv_batch* batch, const int32_t* kv_lens, int32_t max_kv_len,
                                 int32_t window, const void* q, float softmax_scale,
                                 void* out, int32_t out_dtype, float* lse,
                                 int32_t* status_flags, void* stream);

/* Chunked-prefill attention (Sections 3.4, 3.5): the new phase's queries over the cached Q4
 * prefix plus the causal new tokens, which must already have been appended (they are read
 * back in quantized form, so the result does not depend on the chunk size).
 *   kv_lens [A]    total keys including the new chunk
 *   q_offs  [A+1]  prefix sums of query counts; q_len[a] = q_offs[a+1]-q_offs[a]; query i of
 *                  agent a sits at position kv_len-q_len+i and attends keys j <= position
 *                  (and j > position - window when window > 0)
 *   total_q, max_q_len, max_kv_len   host copies / upper bounds (size the grid)
 *   q bf16 [total_q][n_q_heads][d_qk];  out [total_q][n_q_heads][d_v];  lse optional
 *   workspace  at least q4kv_workspace_bytes(spec, A, max_kv_len, total_q) bytes
 * Accuracy: see "Accuracy of the attention entry points" above (spec->exact_products selects
 * between the binary16-tile kernel and the kernel that multiplies the codes). */
int q4kv_prefill_attention(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer,
                           const q4kv_batch* batch, const int32_t* kv_lens, const int32_t* q_offs,
                           int32_t total_q, int32_t max_q_len, int32_t max_kv_len,
                           int32_t window, const void* q, float softmax_scale,
                           void* out, int32_t out_dtype, float* lse,
                           void* workspace, size_t workspace_bytes,
                           int32_t* status_flags, void* stream);

/* Pack: gather one agent's blocks, all layers, through its block-table row into the persisted
 * layout (Appendix A, groups along head_dim): layer outermost, then logical block, then
 *   K_codes u32 [Hkv][256][d_qk/8] | K_scales f16 [Hkv][256][d_qk/64] | K_biases f16 [same] |
 *   V_codes u32 [Hkv][256][d_v/8]  | V_scales f16 [Hkv][256][d_v/64]  | V_biases f16 [same]
 * (no V tensors when v_aliases_k); eight codes per uint32, element k in bits [4k,4k+4).
 * Slots at or beyond n_tokens are written as zero bytes.  dst_bytes must be at least
 * q4kv_packed_bytes(spec, n_tokens).  block_table_row: device, ceil(n_tokens/256) entries. */
int q4kv_pack(const q4kv_spec* spec, const void* pool, int32_t n_blocks,
              const int32_t* block_table_row, int32_t n_tokens,
              void* dst, size_t dst_bytes, int32_t* status_flags, void* stream);

/* Unpack: the inverse scatter, from a persisted buffer into the caller-chosen blocks. */
int q4kv_unpack(const q4kv_spec* spec, const void* src, size_t src_bytes, int32_t n_tokens,
                void* pool, int32_t n_blocks, const int32_t* block_table_row,
                int32_t* status_flags, void* stream);


/* ---- Persisted container and warm restore (Appendix "safetensors Q4 Format"; Section 3.2: the cache is persisted in
 * its quantized form and restored without a dequantize step; the warm-cache rows of the time-to-first-token table) ----
 *
 * One agent's cache as a safetensors file: 8 bytes holding the little-endian length N of the header, N bytes of JSON,
 * then the data section, which is exactly the buffer q4kv_pack writes.  The header lists, layer by layer and block by
 * block, the tensors  L{l}_B{b}_K_weights (U32 [Hkv][256][d_qk/8]), L{l}_B{b}_K_scales, L{l}_B{b}_K_biases
 * (F16 [Hkv][256][d_qk/64]) and the three V tensors likewise (absent when V aliases K), each with its byte range, and
 * carries the spec and the token count under "__metadata__".  The text is canonical: the same cache gives the same
 * bytes, and any safetensors reader can open the file.  All three calls below are host-only. */
size_t q4kv_container_header_bytes(const q4kv_spec* spec, int32_t n_tokens);   /* 8 + N, a multiple of 64; 0: unsupported */
/* dst: HOST memory of at least q4kv_container_header_bytes. */
int q4kv_container_write_header(const q4kv_spec* spec, int32_t n_tokens, void* dst, size_t dst_bytes);
/* src: HOST memory holding at least the header of a container written by this library (any other header is refused
 * with Q4KV_EINVAL).  Returns the spec, the token count and the offset of the data section. */
int q4kv_container_read_header(const void* src, size_t src_bytes, q4kv_spec* spec, int32_t* n_tokens, size_t* data_offset);

/* Save: header into host_image (written at once by the calling thread), then q4kv_pack into dev_staging and one
 * device-to-host copy of the packed bytes behind the header, both enqueued on `stream`.  After the stream has run them,
 * host_image[0 .. header + packed) is the file.  dev_staging: DEVICE, at least q4kv_packed_bytes; host_image: HOST
 * (pinned memory for a copy that overlaps other work), at least q4kv_container_header_bytes + q4kv_packed_bytes. */
int q4kv_save(const q4kv_spec* spec, const void* pool, int32_t n_blocks, const int32_t* block_table_row, int32_t n_tokens,
              void* dev_staging, size_t dev_staging_bytes, void* host_image, size_t host_image_bytes,
              int32_t* status_flags, void* stream);

/* Warm restore: the data section of a container, in HOST memory (pinned, 16-byte aligned), goes to the caller-chosen
 * blocks of the pool in chunks of whole layers: one host-to-device copy per chunk on copy_stream, q4kv_unpack of that
 * chunk on unpack_stream, the copy of the next chunk overlapping the scatter of this one.  dev_staging: DEVICE, at
 * least one layer's packed bytes (q4kv_packed_bytes / n_layers); two layers' worth or more lets copies and scatters
 * overlap.  The two streams may be the same.  The pool is complete when unpack_stream has run everything enqueued here;
 * the call creates and destroys four CUDA events and allocates no memory. */
int q4kv_restore(const q4kv_spec* spec, const void* host_packed, size_t packed_bytes, int32_t n_tokens, void* pool,
                 int32_t n_blocks, const int32_t* block_table_row, void* dev_staging, size_t dev_staging_bytes,
                 int32_t* status_flags, void* copy_stream, void* unpack_stream);

/* ---- Block pool bookkeeping (Section 3.1 "Block Pool with Per-Agent Isolation") ----
 * Host-side policy only; no device memory is touched.  Every block belongs to at most one agent (isolation); agents
 * are kept in least-recently-used order.  When q4kv_allocator_reserve reports Q4KV_EWORKSPACE the pool is full: ask
 * q4kv_allocator_pick_victim for the least recently used agent that is not pinned, persist it (q4kv_save), release
 * it, and reserve again.  Not thread-safe: serialise the calls on one allocator. */
typedef struct q4kv_allocator q4kv_allocator;
q4kv_allocator* q4kv_allocator_create(int32_t n_blocks);            /* NULL: n_blocks <= 0 or no host memory */
void q4kv_allocator_destroy(q4kv_allocator* allocator);
int32_t q4kv_allocator_free_blocks(const q4kv_allocator* allocator);
int32_t q4kv_allocator_agent_blocks(const q4kv_allocator* allocator, int64_t agent_id);   /* 0: unknown agent */
/* Make the agent's block list cover n_tokens (it only grows; earlier blocks keep their place), mark the agent most
 * recently used, and write its block-table row to table_row (HOST, max_blocks entries, -1 past the last block). */
int q4kv_allocator_reserve(q4kv_allocator* allocator, int64_t agent_id, int32_t n_tokens, int32_t* table_row,
                           int32_t max_blocks);
int q4kv_allocator_touch(q4kv_allocator* allocator, int64_t agent_id);                    /* most recently used */
int q4kv_allocator_pin(q4kv_allocator* allocator, int64_t agent_id, int32_t pinned);      /* pinned agents are never victims */
int q4kv_allocator_pick_victim(const q4kv_allocator* allocator, int64_t* agent_id);       /* Q4KV_EWORKSPACE: none */
int q4kv_allocator_release(q4kv_allocator* allocator, int64_t agent_id);                  /* its blocks become free */

/* ---- Dense-batch shim (Section 3.4: BatchQuantizedKVCache.merge / extract) ----
 * The paper stacks caches of different lengths into one left-padded batch.  This library attends through block tables
 * and needs no such copy; these two calls serve code that holds, or wants, the dense form of ONE layer:
 *   K_codes u32 [A][Hkv][T][d_qk/8] | K_scales f16 [A][Hkv][T][d_qk/64] | K_biases | V_codes | V_scales | V_biases
 * (no V tensors when v_aliases_k), one tensor after the other, agent a's kv_lens[a] tokens in rows T - kv_lens[a] ..
 * T - 1 and zero bytes in the padding rows before them.  merge: dense -> the agents' pool blocks (cache positions
 * 0 .. kv_lens[a] - 1); extract: the reverse.  kv_lens: DEVICE [A]; a length above T or above max_blocks * 256 raises
 * Q4KV_FLAG_BAD_LENGTH and skips the agent.  dense: DEVICE, at least q4kv_dense_bytes(spec, A, T). */
size_t q4kv_dense_bytes(const q4kv_spec* spec, int32_t n_agents, int32_t T);
int q4kv_merge_dense(const q4kv_spec* spec, void* pool, int32_t n_blocks, int32_t layer, const q4kv_batch* batch,
                     const int32_t* kv_lens, int32_t T, const void* dense, size_t dense_bytes, int32_t* status_flags,
                     void* stream);
int q4kv_extract_dense(const q4kv_spec* spec, const void* pool, int32_t n_blocks, int32_t layer, const q4kv_batch* batch,
                       const int32_t* kv_lens, int32_t T, void* dense, size_t dense_bytes, int32_t* status_flags,
                       void* stream);

#ifdef __cplusplus
}
#endif
#endif /* Q4KV_H */
