// paged_decode_reduce: merge split-KV partials by their log-sum-exp weights.
// One warp per (sequence, query token, query head) row; a lane owns 4 (or, for head_dim 256, 8) output
// columns. The chunks' log-sum-exps are read once, one per lane, and turned into weights that stay in
// registers; the accumulation then broadcasts a weight by shuffle and reads the chunk's partial row
// with one coalesced 16-byte load per lane, all loads independent of one another (a thread per column
// looping over the chunks waited for one L2 access after the other).
#include "common.cuh"

namespace pda {

namespace {
constexpr int kReduceWarps = 4;       // rows per CTA
constexpr int kReduceMaxBlocks = 8;   // weights held in registers: up to 8 x 32 chunks, more are recomputed
}  // namespace

__global__ void __launch_bounds__(kReduceWarps * 32)
reduce_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
              const int32_t* __restrict__ seq_lens, int32_t num_q_heads, int32_t head_dim,
              int32_t chunk_tokens, int32_t max_chunks, int32_t first_token, int32_t first_chunks,
              int32_t tokens_per_seq, int64_t n_rows, __nv_bfloat16* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * kReduceWarps + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int b = static_cast<int>(row / (static_cast<int64_t>(tokens_per_seq) * num_q_heads));  // row = (b, token, head)
  // first_chunks fixed slots (a shared prefix computed once), then the chunks of [first_token, L)
  const int L = max(seq_lens[b] - first_token, 0);
  int n_chunks = first_chunks + (L + chunk_tokens - 1) / chunk_tokens;
  n_chunks = min(n_chunks, max_chunks);
  const float* lse = part_lse + row * max_chunks;
  float M = -INFINITY;
  for (int c = lane; c < n_chunks; c += 32) M = fmaxf(M, lse[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float wreg[kReduceMaxBlocks];
  float W = 0.f;
#pragma unroll
  for (int k = 0; k < kReduceMaxBlocks; ++k) {
    const int c = k * 32 + lane;
    wreg[k] = (c < n_chunks && M > -INFINITY) ? __expf(lse[c] - M) : 0.f;
    W += wreg[k];
  }
  for (int c = kReduceMaxBlocks * 32 + lane; c < n_chunks; c += 32) W += M > -INFINITY ? __expf(lse[c] - M) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) W += __shfl_xor_sync(0xffffffffu, W, o);
  const float inv = W > 0.f ? 1.f / W : 0.f;
  const int vecs = head_dim / 4;  // 16-byte vectors per row
  const float4* po = reinterpret_cast<const float4*>(part_o + row * max_chunks * head_dim);
  for (int v0 = 0; v0 < vecs; v0 += 32) {
    const int v = v0 + lane;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int k = 0; k < kReduceMaxBlocks; ++k) {
      if (k * 32 >= n_chunks) break;  // warp-uniform
      const int n_here = min(32, n_chunks - k * 32);
#pragma unroll 8
      for (int cc = 0; cc < n_here; ++cc) {
        const float w = __shfl_sync(0xffffffffu, wreg[k], cc);
        if (v < vecs) {
          const float4 x = __ldg(po + static_cast<int64_t>(k * 32 + cc) * vecs + v);
          acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y);
          acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
        }
      }
    }
    for (int c = kReduceMaxBlocks * 32; c < n_chunks; ++c) {  // (more than 256 chunks: weights recomputed)
      const float w = M > -INFINITY ? __expf(lse[c] - M) : 0.f;  // (every chunk empty: zeros, as above)
      if (v < vecs) {
        const float4 x = __ldg(po + static_cast<int64_t>(c) * vecs + v);
        acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y);
        acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
      }
    }
    if (v < vecs) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
      __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
      uint2 packed;
      packed.x = *reinterpret_cast<uint32_t*>(&lo);
      packed.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(out + row * head_dim + 4 * v) = packed;
    }
  }
}

// The same merge with a CTA per row, its four warps sharing the row's chunks (warp w takes chunks w, w + 4,
// ...) and adding their sums in a fixed order through shared memory: for launches with few rows and many
// chunks (a long-context batch: 256 rows of 60 chunks), where a warp per row leaves most SMs idle and walks
// its chunks alone (16.7 us measured on 64 rows x 70 chunks).
__global__ void __launch_bounds__(kReduceWarps * 32)
reduce_row_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                  const int32_t* __restrict__ seq_lens, int32_t num_q_heads, int32_t head_dim,
                  int32_t chunk_tokens, int32_t max_chunks, int32_t first_token, int32_t first_chunks,
                  int32_t tokens_per_seq, __nv_bfloat16* __restrict__ out) {
  __shared__ float4 part_sh[kReduceWarps][64];  // [warp][16-byte vector of the row], head_dim <= 256
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t row = blockIdx.x;
  const int b = static_cast<int>(row / (static_cast<int64_t>(tokens_per_seq) * num_q_heads));
  const int L = max(seq_lens[b] - first_token, 0);
  int n_chunks = first_chunks + (L + chunk_tokens - 1) / chunk_tokens;
  n_chunks = min(n_chunks, max_chunks);
  const float* lse = part_lse + row * max_chunks;
  // every warp computes the row's maximum and weight sum the same way (same values in all four)
  float M = -INFINITY;
  for (int c = lane; c < n_chunks; c += 32) M = fmaxf(M, lse[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float W = 0.f;
  for (int c = lane; c < n_chunks; c += 32) W += M > -INFINITY ? __expf(lse[c] - M) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) W += __shfl_xor_sync(0xffffffffu, W, o);
  const float inv = W > 0.f ? 1.f / W : 0.f;
  const int vecs = head_dim / 4;
  const float4* po = reinterpret_cast<const float4*>(part_o + row * max_chunks * head_dim);
  for (int v0 = 0; v0 < vecs; v0 += 32) {
    const int v = v0 + lane;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (v < vecs) {
#pragma unroll 4
      for (int c = warp; c < n_chunks; c += kReduceWarps) {
        const float w = M > -INFINITY ? __expf(__ldg(lse + c) - M) : 0.f;
        const float4 x = __ldg(po + static_cast<int64_t>(c) * vecs + v);
        acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y);
        acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
      }
      part_sh[warp][v] = acc;
    }
  }
  __syncthreads();
  for (int v = threadIdx.x; v < vecs; v += kReduceWarps * 32) {
    float4 acc = part_sh[0][v];
#pragma unroll
    for (int w = 1; w < kReduceWarps; ++w) {
      const float4 x = part_sh[w][v];
      acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + row * head_dim + 4 * v) = packed;
  }
}

cudaError_t launch_reduce(const float* part_o, const float* part_lse, const int32_t* seq_lens,
                          int32_t batch, int32_t num_q_heads, int32_t head_dim,
                          int32_t chunk_tokens, int32_t max_chunks, int32_t first_token,
                          int32_t first_chunks, int32_t tokens_per_seq, __nv_bfloat16* out,
                          cudaStream_t stream) {
  if (batch == 0 || num_q_heads == 0 || tokens_per_seq == 0) return cudaSuccess;
  const int64_t n_rows = static_cast<int64_t>(batch) * tokens_per_seq * num_q_heads;
  const int64_t blocks = (n_rows + kReduceWarps - 1) / kReduceWarps;
  if (blocks > INT32_MAX) return cudaErrorInvalidValue;
  if (n_rows <= 1024 && max_chunks >= 8 && head_dim <= 256) {  // few rows, many chunks: a CTA per row
    reduce_row_kernel<<<static_cast<unsigned>(n_rows), kReduceWarps * 32, 0, stream>>>(
        part_o, part_lse, seq_lens, num_q_heads, head_dim, chunk_tokens, max_chunks, first_token,
        first_chunks, tokens_per_seq, out);
    return cudaGetLastError();
  }
  reduce_kernel<<<static_cast<unsigned>(blocks), kReduceWarps * 32, 0, stream>>>(
      part_o, part_lse, seq_lens, num_q_heads, head_dim, chunk_tokens, max_chunks, first_token,
      first_chunks, tokens_per_seq, n_rows, out);
  return cudaGetLastError();
}

}  // namespace pda
