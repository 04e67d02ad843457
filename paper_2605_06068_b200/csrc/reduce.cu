// paged_decode_reduce: merge split-KV partials by their log-sum-exp weights.
// One CTA per (sequence, query head); thread d owns output element d.
#include "common.cuh"

namespace pda {

__global__ void reduce_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                              const int32_t* __restrict__ seq_lens, int32_t num_q_heads,
                              int32_t head_dim, int32_t chunk_tokens, int32_t max_chunks,
                              int32_t first_token, int32_t first_chunks, int32_t tokens_per_seq,
                              __nv_bfloat16* __restrict__ out) {
  const int h = blockIdx.x;
  const int b = blockIdx.y / tokens_per_seq;  // blockIdx.y = sequence * tokens_per_seq + query token
  const int64_t row = static_cast<int64_t>(blockIdx.y) * num_q_heads + h;
  // first_chunks fixed slots (a shared prefix computed once), then the chunks of [first_token, L)
  const int L = max(seq_lens[b] - first_token, 0);
  int n_chunks = first_chunks + (L + chunk_tokens - 1) / chunk_tokens;
  n_chunks = min(n_chunks, max_chunks);
  const float* lse = part_lse + row * max_chunks;
  float M = -INFINITY;
  for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, lse[c]);
  for (int d = threadIdx.x; d < head_dim; d += blockDim.x) {
    float acc = 0.f, W = 0.f;
    if (M > -INFINITY) {
      const float* po = part_o + row * max_chunks * head_dim + d;
      for (int c = 0; c < n_chunks; ++c) {
        const float w = __expf(lse[c] - M);
        W += w;
        acc = fmaf(w, po[static_cast<int64_t>(c) * head_dim], acc);
      }
      acc /= W;
    }
    out[row * head_dim + d] = __float2bfloat16_rn(acc);
  }
}

cudaError_t launch_reduce(const float* part_o, const float* part_lse, const int32_t* seq_lens,
                          int32_t batch, int32_t num_q_heads, int32_t head_dim,
                          int32_t chunk_tokens, int32_t max_chunks, int32_t first_token,
                          int32_t first_chunks, int32_t tokens_per_seq, __nv_bfloat16* out,
                          cudaStream_t stream) {
  if (batch == 0 || num_q_heads == 0 || tokens_per_seq == 0) return cudaSuccess;
  dim3 grid(num_q_heads, batch * tokens_per_seq);
  const int threads = head_dim <= 128 ? 128 : 256;
  reduce_kernel<<<grid, threads, 0, stream>>>(part_o, part_lse, seq_lens, num_q_heads, head_dim,
                                              chunk_tokens, max_chunks, first_token, first_chunks, tokens_per_seq, out);
  return cudaGetLastError();
}

}  // namespace pda
