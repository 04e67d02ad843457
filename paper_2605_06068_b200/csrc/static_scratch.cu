// paged_decode_attention_static: split-KV attention + reduce whose partial
// buffers live in a fixed device array owned by the library, for callers that
// cannot obtain device memory of their own at call time.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = PDA_STATIC_SCRATCH_BYTES;

// Scratch for the split-KV partials. File-scope device storage: a device carries
// these bytes from the moment this file's device image is loaded on it (the
// runtime loads images lazily, so that is the first address lookup below) until
// the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device. In host code the
// symbol's name is only a handle, so the address is looked up once per device
// (with that device current) and cached. The first lookup on a device loads the
// image and can fail (no room left for the array): the error is returned, and
// nothing is cached, so a later call tries again.
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int paged_decode_attention_static(
    const void* q, const void* k_cache, const void* v_cache, const pda_cache_desc* desc,
    const float* k_scale, const float* v_scale, const int32_t* block_table,
    int32_t block_table_stride, const int32_t* seq_lens, int32_t batch, int32_t num_q_heads,
    float scale, int32_t chunk_tokens, int32_t max_chunks, void* out, int32_t* status,
    pda_stream_t stream) {
  if (desc == nullptr || out == nullptr) return PDA_ERR_INVALID_ARG;
  if (chunk_tokens <= 0 || max_chunks <= 0 || batch < 0 || num_q_heads <= 0 || desc->head_dim <= 0)
    return PDA_ERR_INVALID_ARG;
  // part_o [B,Hq,C,D] fp32 followed (256-byte aligned) by part_lse [B,Hq,C] fp32
  const size_t rows = static_cast<size_t>(batch) * num_q_heads * max_chunks;
  const size_t o_bytes = (rows * desc->head_dim * 4 + 255) & ~static_cast<size_t>(255);
  const size_t need = o_bytes + rows * 4;
  if (need > kScratchBytes) return PDA_ERR_TOO_LARGE;
  // (before the empty-batch return: a start-up call with batch 0 is how a caller gets the image that holds
  // the array loaded, and its bytes reserved, while the device still has room)
  void* base = nullptr;
  if (cudaError_t e = scratch_address(&base)) return static_cast<int>(e);
  if (batch == 0) return PDA_OK;
  float* part_o = static_cast<float*>(base);
  float* part_lse = reinterpret_cast<float*>(static_cast<unsigned char*>(base) + o_bytes);
  if (int rc = paged_decode_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                                      block_table_stride, seq_lens, batch, num_q_heads, scale,
                                      chunk_tokens, nullptr, part_o, part_lse, max_chunks, 0u,
                                      status, stream))
    return rc;
  return paged_decode_reduce(part_o, part_lse, seq_lens, batch, num_q_heads, desc->head_dim,
                             chunk_tokens, max_chunks, out, stream);
}
