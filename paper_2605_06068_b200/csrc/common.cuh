// Shared device helpers and the internal launcher interface of libpda.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pda.h"

namespace pda {

constexpr int kPageSize = 16;

// Geometry handed to every kernel by value.
struct CacheGeom {
  int64_t page_stride, head_stride, slot_stride;  // elements
  int32_t num_pages, num_kv_heads, head_dim, dtype;
};

struct AttnParams {
  const __nv_bfloat16* q;
  const void* k_cache;
  const void* v_cache;
  const float* k_scale;
  const float* v_scale;
  const int32_t* block_table;
  const int32_t* seq_lens;
  __nv_bfloat16* out;
  float* part_o;
  float* part_lse;
  int32_t* status;
  CacheGeom geom;
  int32_t block_table_stride, batch, num_q_heads, group;  // group = Hq / Hkv
  int32_t chunk_tokens, max_chunks;
  float scale;
  // Token range: tokens below max(first_token, L - window) are not attended (window <= 0: no
  // window). Chunk c covers [first_token + c*chunk_tokens, ...) and is stored in partial slot
  // chunk_slot0 + c. first_token is a multiple of the page size.
  int32_t window, first_token, chunk_slot0;
};

// Fused decode step (attention_tma.cu): attention parameters plus the
// optional append inputs, the optional workspace and the reduce switch.
struct StepParams {
  AttnParams a;
  const void* k_new;   // [B,Hkv,D] bf16 or nullptr (no append)
  const void* v_new;
  void* k_cache_w;     // writable aliases of a.k_cache / a.v_cache (append target)
  void* v_cache_w;
  int32_t* workspace;  // per-(sequence, kv head) chunk counters at [2 ..); nullptr when nothing is counted
  int32_t fuse_reduce; // 1: the launch writes `out` itself (needs workspace when split)
};

// Multi-query attention (attention_mq.cu): n_q query tokens per sequence.
struct MqParams {
  AttnParams a;           // q is [B, n_q, Hq, D]; out / partials are indexed by (b*n_q + i)
  int32_t n_q;            // query tokens per sequence
  int32_t causal;         // 1: query i sees keys j < L - n_q + i + 1
  int32_t kv_len_fixed;   // > 0: every sequence attends [first_token, kv_len_fixed) (shared prefix)
  int32_t n_chunks_grid;  // chunk CTAs launched per (sequence, head) when split
};

__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status != nullptr) atomicMax(status, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t bits) {
  return __uint_as_float(static_cast<uint32_t>(bits) << 16);
}

// E4M3 byte -> float from the bit fields: exponent 0 is subnormal (m * 2^-9),
// S.1111.111 is NaN, everything else (1 + m/8) * 2^(e-7).
__device__ __forceinline__ float e4m3_to_float(uint8_t byte) {
  const uint32_t sign = static_cast<uint32_t>(byte & 0x80) << 24;
  const uint32_t e = (byte >> 3) & 0xF;
  const uint32_t m = byte & 0x7;
  uint32_t bits;
  if (e == 0xF && m == 0x7) {
    bits = 0x7FC00000u;
  } else if (e == 0) {
    bits = __float_as_uint(static_cast<float>(m) * 0.001953125f);
  } else {
    bits = ((e + 120u) << 23) | (m << 20);
  }
  return __uint_as_float(bits | sign);
}

// Launchers (each returns the cudaError_t of its launch).
cudaError_t launch_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                             const CacheGeom& g, const int32_t* block_table, int32_t bt_stride,
                             const int32_t* seq_lens, int32_t batch, int32_t* status,
                             cudaStream_t stream);
cudaError_t launch_kv_append_e4m3(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                  float* k_scale, float* v_scale, const CacheGeom& g,
                                  const int32_t* block_table, int32_t bt_stride,
                                  const int32_t* seq_lens, int32_t batch, int32_t n_new, int32_t* status,
                                  cudaStream_t stream);
cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int32_t batch, int32_t delta, cudaStream_t stream);
// table_host / lens_host: device addresses of pinned, mapped host memory
cudaError_t launch_stage_tables(const int32_t* table_host, int32_t* table_dev, int64_t n_table,
                                const int32_t* lens_host, int32_t* lens_dev, int32_t batch, cudaStream_t stream);
cudaError_t launch_attention_generic(const AttnParams& p, cudaStream_t stream);
// Returns cudaErrorNotSupported when the shape is outside the fast kernel's set.
cudaError_t launch_attention_tma(const AttnParams& p, cudaStream_t stream);
bool attention_tma_supports(const AttnParams& p);
// Fused step on the same kernel: optional append, optional in-kernel reduce (sp.fuse_reduce).
cudaError_t launch_step_tma(const StepParams& sp, cudaStream_t stream);
// Persistent form of the fused step for unsplit launches (needs the workspace's work ticket).
bool attention_persist_supports(const StepParams& sp);
bool attention_persist_preferred(const StepParams& sp, int min_units_per_cta);
cudaError_t launch_attention_persist(const StepParams& sp, cudaStream_t stream);
// Rows are (sequence, query token, head): tokens_per_seq query tokens share one seq_lens entry.
cudaError_t launch_reduce(const float* part_o, const float* part_lse, const int32_t* seq_lens,
                          int32_t batch, int32_t num_q_heads, int32_t head_dim,
                          int32_t chunk_tokens, int32_t max_chunks, int32_t first_token,
                          int32_t first_chunks, int32_t tokens_per_seq, __nv_bfloat16* out,
                          cudaStream_t stream);
bool attention_mq_supports(const MqParams& mp);
// tcgen05 + TMEM version (bf16 KV, head_dim 128)
bool attention_mq_tc_supports(const MqParams& mp);
cudaError_t launch_attention_mq_tc(const MqParams& mp, cudaStream_t stream);
bool attention_mq_tcp_supports(const MqParams& mp);
cudaError_t launch_attention_mq_tcp(const MqParams& mp, cudaStream_t stream);
// persistent tcgen05 + TMEM version for e4m3 KV (head_dim 128, unsplit)
bool attention_mq_tc8p_supports(const MqParams& mp);
cudaError_t launch_attention_mq_tc8p(const MqParams& mp, cudaStream_t stream);
cudaError_t launch_attention_mq(const MqParams& mp, cudaStream_t stream);
cudaError_t launch_kv_append_tokens(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                    const CacheGeom& g, const int32_t* block_table, int32_t bt_stride,
                                    const int32_t* seq_lens, int32_t batch, int32_t n_new,
                                    int32_t* status, cudaStream_t stream);
cudaError_t launch_e4m3_decode(float* out256, cudaStream_t stream);
cudaError_t launch_wait_timeout(uint32_t polls, int32_t* status, uint64_t* result, cudaStream_t stream);
cudaError_t launch_read_probe(const void* buf, size_t bytes, uint32_t* sink, cudaStream_t stream);

}  // namespace pda
