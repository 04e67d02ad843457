// Generic paged decode attention on CUDA cores: any group size, any head_dim
// that is a multiple of 32 up to 256, any cache strides, bf16 or e4m3 KV.
// One warp per (sequence, query head, chunk). It is the simple path for shapes
// outside the TMA + tensor-core kernel and the in-library cross-check for it.
//
// Per tile of 32 tokens: lane j scores token j (fp32 dot over head_dim), the
// warp takes max and sum by shuffles, then each lane accumulates its own
// head_dim/32 output columns over the tile's tokens.
#include "common.cuh"

namespace pda {

namespace {

constexpr int kMaxDPerLane = 8;  // head_dim <= 256

template <bool kFp8>
__device__ __forceinline__ float load_elem(const void* base, int64_t idx) {
  if (kFp8) return e4m3_to_float(static_cast<const uint8_t*>(base)[idx]);
  return bf16_bits_to_float(static_cast<const uint16_t*>(base)[idx]);
}

template <bool kFp8>
__global__ void __launch_bounds__(32) attention_generic_kernel(AttnParams p) {
  const int lane = threadIdx.x;
  const int c = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int D = p.geom.head_dim;
  const int g = h / p.group;
  const int64_t row = static_cast<int64_t>(b) * p.num_q_heads + h;
  const bool split = p.chunk_tokens > 0;

  const int L = max(p.seq_lens[b], 0);
  int t0 = p.first_token, t1 = L;
  if (split) {
    t0 = p.first_token + c * p.chunk_tokens;
    if (t0 >= L) return;  // no such chunk
    t1 = min(t0 + p.chunk_tokens, L);
  }
  // window: tokens before L - window are not attended; the unit may end up empty
  if (p.window > 0 && L - p.window > t0) t0 = min(L - p.window, t1);
  const bool too_long =
      static_cast<int64_t>(L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ||
      (split && static_cast<int64_t>(L - p.first_token) >
                    static_cast<int64_t>(p.max_chunks - p.chunk_slot0) * p.chunk_tokens);

  __shared__ float q_s[256];
  for (int d = lane; d < D; d += 32) q_s[d] = __bfloat162float(p.q[row * D + d]);
  __syncwarp();

  float m = -INFINITY, l = 0.f;
  float acc[kMaxDPerLane];
#pragma unroll
  for (int i = 0; i < kMaxDPerLane; ++i) acc[i] = 0.f;
  bool bad_page = false;
  const int32_t* table = p.block_table + static_cast<int64_t>(b) * p.block_table_stride;

  for (int base = t0; base < t1 && !too_long; base += 32) {
    // ---- scores: lane j <-> token base + j
    const int j = base + lane;
    const bool valid = j < t1;
    int page = 0;
    if (valid) {
      page = table[j / kPageSize];
      if (page < 0 || page >= p.geom.num_pages) bad_page = true;
    }
    if (__any_sync(0xffffffffu, bad_page)) { bad_page = true; break; }
    float s = -INFINITY;
    if (valid) {
      const int64_t off = page * p.geom.page_stride + g * p.geom.head_stride +
                          (j % kPageSize) * p.geom.slot_stride;
      float dot = 0.f;
      for (int d = 0; d < D; ++d) dot = fmaf(q_s[d], load_elem<kFp8>(p.k_cache, off + d), dot);
      if (kFp8) dot *= p.k_scale[static_cast<int64_t>(page) * p.geom.num_kv_heads + g];
      s = dot * p.scale;
    }
    // ---- online softmax update
    float tile_max = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tile_max = fmaxf(tile_max, __shfl_xor_sync(0xffffffffu, tile_max, o));
    const float m_new = fmaxf(m, tile_max);          // finite: the tile has >= 1 valid token
    const float alpha = (m == -INFINITY) ? 0.f : expf(m - m_new);
    float pj = valid ? expf(s - m_new) : 0.f;
    float tile_sum = pj;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tile_sum += __shfl_xor_sync(0xffffffffu, tile_sum, o);
    l = l * alpha + tile_sum;
    m = m_new;
    if (kFp8 && valid) pj *= p.v_scale[static_cast<int64_t>(page) * p.geom.num_kv_heads + g];
#pragma unroll
    for (int i = 0; i < kMaxDPerLane; ++i) acc[i] *= alpha;
    // ---- PV: lane owns columns lane, lane+32, ...
    const int n_tok = min(32, t1 - base);
    for (int t = 0; t < n_tok; ++t) {
      const float pt = __shfl_sync(0xffffffffu, pj, t);
      const int pg = __shfl_sync(0xffffffffu, page, t);
      const int64_t off = pg * p.geom.page_stride + g * p.geom.head_stride +
                          ((base + t) % kPageSize) * p.geom.slot_stride;
#pragma unroll
      for (int i = 0; i < kMaxDPerLane; ++i) {
        const int d = lane + 32 * i;
        if (d < D) acc[i] = fmaf(pt, load_elem<kFp8>(p.v_cache, off + d), acc[i]);
      }
    }
  }

  const bool failed = bad_page || too_long;
  if (failed && lane == 0) report(p.status, too_long ? PDA_DEV_BAD_SEQ_LEN : PDA_DEV_BAD_PAGE);
  const float inv_l = (l > 0.f && !failed) ? 1.f / l : 0.f;
  if (split) {
    const int64_t pr = row * p.max_chunks + p.chunk_slot0 + c;
    if (p.chunk_slot0 + c >= p.max_chunks) return;
#pragma unroll
    for (int i = 0; i < kMaxDPerLane; ++i) {
      const int d = lane + 32 * i;
      if (d < D) p.part_o[pr * D + d] = failed ? 0.f : acc[i] * inv_l;
    }
    if (lane == 0) p.part_lse[pr] = (l > 0.f && !failed) ? m + logf(l) : -INFINITY;
  } else {
#pragma unroll
    for (int i = 0; i < kMaxDPerLane; ++i) {
      const int d = lane + 32 * i;
      if (d < D) p.out[row * D + d] = __float2bfloat16_rn(failed ? 0.f : acc[i] * inv_l);
    }
  }
}

}  // namespace

cudaError_t launch_attention_generic(const AttnParams& p, cudaStream_t stream) {
  if (p.batch == 0 || p.num_q_heads == 0) return cudaSuccess;
  const unsigned chunks = p.chunk_tokens > 0 ? static_cast<unsigned>(p.max_chunks - p.chunk_slot0) : 1u;
  dim3 grid(chunks, p.num_q_heads, p.batch);
  if (p.geom.dtype == PDA_FP8_E4M3)
    attention_generic_kernel<true><<<grid, 32, 0, stream>>>(p);
  else
    attention_generic_kernel<false><<<grid, 32, 0, stream>>>(p);
  return cudaGetLastError();
}

__global__ void e4m3_decode_kernel(float* out) { out[threadIdx.x] = e4m3_to_float(static_cast<uint8_t>(threadIdx.x)); }

cudaError_t launch_e4m3_decode(float* out256, cudaStream_t stream) {
  e4m3_decode_kernel<<<1, 256, 0, stream>>>(out256);
  return cudaGetLastError();
}

}  // namespace pda
