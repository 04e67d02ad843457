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

// Quantising append into an e4m3 cache: one warp per (sequence, kv head, K|V). The page's
// scale is fixed by its first row (amax * 2 / 448, or 1 for an all-zero row); later rows reuse
// it and saturate at +-448. x / scale is an IEEE fp32 division, the cast rounds to nearest even.
// One warp per (sequence, kv head, K | V) walks the block's n_new tokens in order, so that a page opened
// inside the block gets its scale from the block's own row in slot 0 before the later rows use it (the
// scale of the page being filled stays in a register; a page opened by an earlier call is read once).
__global__ void kv_append_e4m3_kernel(const __nv_bfloat16* __restrict__ k_new,
                                      const __nv_bfloat16* __restrict__ v_new,
                                      uint8_t* __restrict__ k_cache, uint8_t* __restrict__ v_cache,
                                      float* __restrict__ k_scale, float* __restrict__ v_scale,
                                      CacheGeom g, const int32_t* __restrict__ block_table,
                                      int32_t bt_stride, const int32_t* __restrict__ seq_lens,
                                      int32_t batch, int32_t n_new, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t unit = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (unit >= 2ll * batch * g.num_kv_heads) return;
  const bool is_v = unit >= static_cast<int64_t>(batch) * g.num_kv_heads;
  const int64_t r = is_v ? unit - static_cast<int64_t>(batch) * g.num_kv_heads : unit;
  const int head = static_cast<int>(r % g.num_kv_heads), b = static_cast<int>(r / g.num_kv_heads);
  const int L = seq_lens[b];
  if (L <= 0) return;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(bt_stride) * kPageSize) {
    if (lane == 0) report(status, PDA_DEV_BAD_SEQ_LEN);
    return;
  }
  const int per_lane = g.head_dim / 32;  // 2, 4, 6 or 8 consecutive elements
  int cur_page = -1;   // the page whose scale `sc` is
  float sc = 1.f;
  for (int i = 0; i < n_new; ++i) {
    const int pos = L - n_new + i;
    if (pos < 0) continue;
    const int page = block_table[static_cast<int64_t>(b) * bt_stride + pos / kPageSize];
    if (page < 0 || page >= g.num_pages) {
      if (lane == 0) report(status, PDA_DEV_BAD_PAGE);
      cur_page = -1;
      continue;
    }
    const int slot = pos % kPageSize;
    const __nv_bfloat16* src = (is_v ? v_new : k_new) +
                               ((static_cast<int64_t>(b) * n_new + i) * g.num_kv_heads + head) * g.head_dim + lane * per_lane;
    float x[8];
    float amax = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      x[e] = e < per_lane ? __bfloat162float(src[e]) : 0.f;
      amax = fmaxf(amax, fabsf(x[e]));
    }
    float* scale_ptr = (is_v ? v_scale : k_scale) + static_cast<int64_t>(page) * g.num_kv_heads + head;
    if (slot == 0) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      sc = amax > 0.f ? __fdiv_rn(amax * 2.0f, 448.0f) : 1.0f;
      if (lane == 0) *scale_ptr = sc;
    } else if (page != cur_page) {
      sc = *scale_ptr;   // opened by an earlier call
    }
    cur_page = page;
    uint8_t* dst = (is_v ? v_cache : k_cache) + page * g.page_stride + head * g.head_stride +
                   slot * g.slot_stride + lane * per_lane;
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      if (e < per_lane) {
        uint16_t packed;
        const float lo = __fdiv_rn(x[e], sc), hi = __fdiv_rn(x[e + 1], sc);
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(packed) : "f"(hi), "f"(lo));
        *reinterpret_cast<uint16_t*>(dst + e) = packed;
      }
    }
  }
}

cudaError_t launch_kv_append_e4m3(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                  float* k_scale, float* v_scale, const CacheGeom& g,
                                  const int32_t* block_table, int32_t bt_stride,
                                  const int32_t* seq_lens, int32_t batch, int32_t n_new, int32_t* status,
                                  cudaStream_t stream) {
  const int64_t warps = 2ll * batch * g.num_kv_heads;
  if (warps == 0 || n_new == 0) return cudaSuccess;
  const int threads = 128;
  const unsigned blocks = static_cast<unsigned>((warps * 32 + threads - 1) / threads);
  kv_append_e4m3_kernel<<<blocks, threads, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
      static_cast<uint8_t*>(k_cache), static_cast<uint8_t*>(v_cache), k_scale, v_scale, g,
      block_table, bt_stride, seq_lens, batch, n_new, status);
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

// Copies the step's block table and sequence lengths from pinned, device-mapped host memory into
// their device buffers with one launch (a thread per int32, reads coalesced over the bus): two small
// cudaMemcpyAsync calls ahead of the step cost more than this kernel does.
__global__ void stage_tables_kernel(const int32_t* __restrict__ table_host, int32_t* __restrict__ table_dev,
                                    int64_t n_table, const int32_t* __restrict__ lens_host,
                                    int32_t* __restrict__ lens_dev, int32_t batch) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n_table) table_dev[i] = table_host[i];
  else if (i - n_table < batch) lens_dev[i - n_table] = lens_host[i - n_table];
}

cudaError_t launch_stage_tables(const int32_t* table_host, int32_t* table_dev, int64_t n_table,
                                const int32_t* lens_host, int32_t* lens_dev, int32_t batch, cudaStream_t stream) {
  const int64_t n = n_table + batch;
  if (n == 0) return cudaSuccess;
  stage_tables_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(table_host, table_dev, n_table,
                                                                               lens_host, lens_dev, batch);
  return cudaGetLastError();
}

}  // namespace pda
