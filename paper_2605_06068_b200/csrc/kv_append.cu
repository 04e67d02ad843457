// kv_append: scatter this step's new key/value rows into their page slots.
// Pure index arithmetic plus 16-byte copies; one thread per 16-byte vector.
#include "common.cuh"

namespace pda {

__global__ void kv_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                 uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                 CacheGeom g, const int32_t* __restrict__ block_table,
                                 int32_t bt_stride, const int32_t* __restrict__ seq_lens,
                                 int32_t batch, int32_t* status) {
  const int vec_per_row = g.head_dim / 8;  // 8 bf16 per 16-byte vector
  const int64_t per_cache = static_cast<int64_t>(batch) * g.num_kv_heads * vec_per_row;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= 2 * per_cache) return;
  const bool is_v = i >= per_cache;
  const int64_t r = is_v ? i - per_cache : i;
  const int vec = static_cast<int>(r % vec_per_row);
  const int head = static_cast<int>((r / vec_per_row) % g.num_kv_heads);
  const int b = static_cast<int>(r / (static_cast<int64_t>(vec_per_row) * g.num_kv_heads));
  const int L = seq_lens[b];
  if (L <= 0) return;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(bt_stride) * kPageSize) {
    report(status, PDA_DEV_BAD_SEQ_LEN);
    return;
  }
  const int page = block_table[static_cast<int64_t>(b) * bt_stride + (L - 1) / kPageSize];
  if (page < 0 || page >= g.num_pages) {
    report(status, PDA_DEV_BAD_PAGE);
    return;
  }
  const int slot = (L - 1) % kPageSize;
  const int64_t dst = (page * g.page_stride + head * g.head_stride + slot * g.slot_stride) / 8 + vec;
  if (is_v) v_cache[dst] = v_new[r]; else k_cache[dst] = k_new[r];
}

cudaError_t launch_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                             const CacheGeom& g, const int32_t* block_table, int32_t bt_stride,
                             const int32_t* seq_lens, int32_t batch, int32_t* status,
                             cudaStream_t stream) {
  const int64_t total = 2ll * batch * g.num_kv_heads * (g.head_dim / 8);
  if (total == 0) return cudaSuccess;
  const int threads = 256;
  const unsigned blocks = static_cast<unsigned>((total + threads - 1) / threads);
  kv_append_kernel<<<blocks, threads, 0, stream>>>(
      static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
      static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), g, block_table, bt_stride,
      seq_lens, batch, status);
  return cudaGetLastError();
}

// n_new tokens per sequence: token i of new[b] goes to logical index L - n_new + i.
__global__ void kv_append_tokens_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                        uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                        CacheGeom g, const int32_t* __restrict__ block_table,
                                        int32_t bt_stride, const int32_t* __restrict__ seq_lens,
                                        int32_t batch, int32_t n_new, int32_t* status) {
  const int vec_per_row = g.head_dim / 8;
  const int64_t per_cache = static_cast<int64_t>(batch) * n_new * g.num_kv_heads * vec_per_row;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= 2 * per_cache) return;
  const bool is_v = i >= per_cache;
  const int64_t r = is_v ? i - per_cache : i;
  const int vec = static_cast<int>(r % vec_per_row);
  const int head = static_cast<int>((r / vec_per_row) % g.num_kv_heads);
  const int tok = static_cast<int>((r / (static_cast<int64_t>(vec_per_row) * g.num_kv_heads)) % n_new);
  const int b = static_cast<int>(r / (static_cast<int64_t>(vec_per_row) * g.num_kv_heads * n_new));
  const int L = seq_lens[b];
  const int pos = L - n_new + tok;
  if (L <= 0 || pos < 0) return;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(bt_stride) * kPageSize) {
    report(status, PDA_DEV_BAD_SEQ_LEN);
    return;
  }
  const int page = block_table[static_cast<int64_t>(b) * bt_stride + pos / kPageSize];
  if (page < 0 || page >= g.num_pages) {
    report(status, PDA_DEV_BAD_PAGE);
    return;
  }
  const int64_t dst = (page * g.page_stride + head * g.head_stride + (pos % kPageSize) * g.slot_stride) / 8 + vec;
  if (is_v) v_cache[dst] = v_new[r]; else k_cache[dst] = k_new[r];
}

cudaError_t launch_kv_append_tokens(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                    const CacheGeom& g, const int32_t* block_table, int32_t bt_stride,
                                    const int32_t* seq_lens, int32_t batch, int32_t n_new,
                                    int32_t* status, cudaStream_t stream) {
  const int64_t total = 2ll * batch * n_new * g.num_kv_heads * (g.head_dim / 8);
  if (total == 0) return cudaSuccess;
  const int threads = 256;
  const unsigned blocks = static_cast<unsigned>((total + threads - 1) / threads);
  kv_append_tokens_kernel<<<blocks, threads, 0, stream>>>(
      static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
      static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), g, block_table, bt_stride,
      seq_lens, batch, n_new, status);
  return cudaGetLastError();
}

__global__ void advance_seq_lens_kernel(int32_t* seq_lens, int32_t batch, int32_t delta) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < batch) seq_lens[b] += delta;
}

cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int32_t batch, int32_t delta, cudaStream_t stream) {
  if (batch == 0) return cudaSuccess;
  advance_seq_lens_kernel<<<(batch + 255) / 256, 256, 0, stream>>>(seq_lens, batch, delta);
  return cudaGetLastError();
}

}  // namespace pda
