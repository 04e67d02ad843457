// fp64 CPU oracle for batched decode attention over a paged KV cache.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition that the
// CUDA library is checked against. Only the test-suite, the smoke check and
// the benchmark's CPU-baseline / reference legs may load it; the product path
// never does. It shares no header, table, helper or constant with the CUDA
// sources: bf16 and e4m3 decoding are re-derived here from the bit layouts.
//
// What is computed (problem statement: attention of one query token per
// sequence over that sequence's cached keys/values, taken in logical token
// order through a block table; the paper's Appendix A, Scenario A names the
// ingredients: a paged KV cache and grouped-query attention with 32 query
// heads sharing 8 key/value heads):
//
//   for sequence b, query head h, kv head g = h / (Hq / Hkv):
//     for j in [t0, t1):  page = block_table[b][j / P], slot = j % P
//        s_j = scale * sum_d q[b,h,d] * K[page,g,slot,d]
//     m = max_j s_j ; p_j = exp(s_j - m) ; l = sum_j p_j
//     out[d] = (sum_j p_j * V[page,g,slot,d]) / l ;  lse = m + log(l)
//
// The unsplit result uses [t0,t1) = [0,L_b). The split-KV form evaluates the
// same thing per chunk c over [c*chunk, min((c+1)*chunk, L_b)) and
// oracle_paged_decode_reduce merges chunks by their log-sum-exp weights,
// which is algebraically the same softmax.
//
// All sums run in logical order j = t0..t1-1 in double precision; `scale` is
// the fp32 value both sides consume, widened to double.
//
// Parity pins (tests/test_oracle_*.py): dense scaled-dot-product attention
// from a library routine on gathered pages, L=1 returns V exactly, equal
// scores return the mean of V, two-token logistic closed form, page-placement
// invariance, convexity, e4m3 table against the bit definition and a library
// cast, quantiser round trip. No function here is "parity unpinned".

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// bfloat16: the upper 16 bits of an IEEE-754 binary32.
inline double bf16_to_double(uint16_t bits) {
  uint32_t u = static_cast<uint32_t>(bits) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}

// OCP 8-bit float E4M3 ("fn" flavour): 1 sign, 4 exponent (bias 7), 3 mantissa
// bits; exponent 0 is subnormal (m * 2^-9); there is no infinity; S.1111.111 is
// NaN; the largest finite magnitude is S.1111.110 = 448.
inline double e4m3_to_double(uint8_t byte) {
  const int sign = byte >> 7;
  const int e = (byte >> 3) & 0xF;
  const int m = byte & 0x7;
  double mag;
  if (e == 0xF && m == 0x7) {
    return std::numeric_limits<double>::quiet_NaN();
  } else if (e == 0) {
    mag = std::ldexp(static_cast<double>(m), -9);
  } else {
    mag = std::ldexp(1.0 + static_cast<double>(m) / 8.0, e - 7);
  }
  return sign ? -mag : mag;
}

struct CacheView {
  const uint8_t* base;
  int dtype;  // 0 = bf16, 1 = e4m3
  int64_t page_stride, head_stride, slot_stride;  // in elements
  const float* scales;  // [num_pages, Hkv] for e4m3, else unused
  int num_kv_heads;

  double at(int64_t page, int g, int slot, int d) const {
    const int64_t idx = page * page_stride + g * head_stride + slot * slot_stride + d;
    if (dtype == 0) {
      uint16_t bits;
      std::memcpy(&bits, base + 2 * idx, 2);
      return bf16_to_double(bits);
    }
    return e4m3_to_double(base[idx]) *
           static_cast<double>(scales[page * num_kv_heads + g]);
  }
};

// Softmax-weighted average of V rows over logical tokens [t0, t1) for one
// (sequence, query head). Writes out[D] and *lse. An empty range gives
// out = 0 and lse = -inf.
void attend_range(const uint16_t* q_row, const CacheView& K, const CacheView& V,
                  const int32_t* table_row, int P, int D, int g, double scale,
                  int64_t t0, int64_t t1, double* out, double* lse) {
  for (int d = 0; d < D; ++d) out[d] = 0.0;
  if (t1 <= t0) {
    *lse = -std::numeric_limits<double>::infinity();
    return;
  }
  const int64_t n = t1 - t0;
  std::vector<double> s(static_cast<size_t>(n));
  double m = -std::numeric_limits<double>::infinity();
  for (int64_t j = t0; j < t1; ++j) {
    const int64_t page = table_row[j / P];
    const int slot = static_cast<int>(j % P);
    double dot = 0.0;
    for (int d = 0; d < D; ++d) dot += bf16_to_double(q_row[d]) * K.at(page, g, slot, d);
    const double sj = scale * dot;
    s[static_cast<size_t>(j - t0)] = sj;
    if (sj > m) m = sj;
  }
  double l = 0.0;
  for (int64_t j = t0; j < t1; ++j) {
    const double p = std::exp(s[static_cast<size_t>(j - t0)] - m);
    s[static_cast<size_t>(j - t0)] = p;
    l += p;
  }
  for (int64_t j = t0; j < t1; ++j) {
    const int64_t page = table_row[j / P];
    const int slot = static_cast<int>(j % P);
    const double p = s[static_cast<size_t>(j - t0)];
    for (int d = 0; d < D; ++d) out[d] += p * V.at(page, g, slot, d);
  }
  for (int d = 0; d < D; ++d) out[d] /= l;
  *lse = m + std::log(l);
}

template <class F>
void parallel_for(int64_t n, int n_threads, F&& body) {
  if (n_threads <= 1 || n <= 1) {
    for (int64_t i = 0; i < n; ++i) body(i);
    return;
  }
  std::atomic<int64_t> next{0};
  std::vector<std::thread> pool;
  for (int t = 0; t < n_threads; ++t) {
    pool.emplace_back([&] {
      for (;;) {
        const int64_t i = next.fetch_add(1);
        if (i >= n) break;
        body(i);
      }
    });
  }
  for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

int oracle_hardware_threads() {
  const unsigned n = std::thread::hardware_concurrency();
  return n == 0 ? 1 : static_cast<int>(n);
}

// table[byte] = value of the e4m3 byte (NaN for 0x7F and 0xFF).
void oracle_e4m3_decode_table(double* table256) {
  for (int i = 0; i < 256; ++i) table256[i] = e4m3_to_double(static_cast<uint8_t>(i));
}

// KV append: the token at logical index L_b - 1 (seq_lens holds the length
// AFTER the append) is copied bytewise into page block_table[b][(L_b-1)/P],
// slot (L_b-1)%P, for every kv head. Sequences with L_b <= 0 append nothing.
// elem_bytes is 2 (bf16 cache). new rows are [B, Hkv, D] contiguous.
void oracle_kv_append(const uint8_t* k_new, const uint8_t* v_new, uint8_t* k_cache,
                      uint8_t* v_cache, int64_t page_stride, int64_t head_stride,
                      int64_t slot_stride, int32_t page_size, int32_t num_kv_heads,
                      int32_t head_dim, int32_t elem_bytes, const int32_t* block_table,
                      int32_t block_table_stride, const int32_t* seq_lens, int32_t batch) {
  for (int b = 0; b < batch; ++b) {
    const int64_t L = seq_lens[b];
    if (L <= 0) continue;
    const int64_t page = block_table[static_cast<int64_t>(b) * block_table_stride + (L - 1) / page_size];
    const int64_t slot = (L - 1) % page_size;
    for (int g = 0; g < num_kv_heads; ++g) {
      const int64_t dst = (page * page_stride + g * head_stride + slot * slot_stride) * elem_bytes;
      const int64_t src = (static_cast<int64_t>(b) * num_kv_heads + g) * head_dim * elem_bytes;
      std::memcpy(k_cache + dst, k_new + src, static_cast<size_t>(head_dim) * elem_bytes);
      std::memcpy(v_cache + dst, v_new + src, static_cast<size_t>(head_dim) * elem_bytes);
    }
  }
}

// Attention. window > 0 restricts every sequence to its last `window` tokens
// (the sliding-window attention of the paper's streaming scenario, Appendix A,
// Scenario D; the definition is the same softmax over that token range).
// chunk_tokens == 0: out is [B,Hq,D], lse is [B,Hq].
// chunk_tokens  > 0: out is [B,Hq,max_chunks,D], lse is [B,Hq,max_chunks];
// entries for chunks c >= ceil(L_b / chunk_tokens) are left untouched.
// kv_dtype: 0 = bf16, 1 = e4m3 with k_scale/v_scale [num_pages,Hkv] fp32.
void oracle_paged_decode_attention(
    const uint16_t* q, const uint8_t* k_cache, const uint8_t* v_cache, int32_t kv_dtype,
    const float* k_scale, const float* v_scale, int64_t page_stride, int64_t head_stride,
    int64_t slot_stride, int32_t page_size, int32_t num_kv_heads, int32_t head_dim,
    const int32_t* block_table, int32_t block_table_stride, const int32_t* seq_lens,
    int32_t batch, int32_t num_q_heads, float scale, int32_t chunk_tokens, int32_t max_chunks,
    int32_t window, double* out, double* lse, int32_t n_threads) {
  const int G = num_q_heads / num_kv_heads;
  const CacheView K{k_cache, kv_dtype, page_stride, head_stride, slot_stride, k_scale, num_kv_heads};
  const CacheView V{v_cache, kv_dtype, page_stride, head_stride, slot_stride, v_scale, num_kv_heads};
  const double sc = static_cast<double>(scale);
  const int64_t rows = static_cast<int64_t>(batch) * num_q_heads;
  parallel_for(rows, n_threads, [&](int64_t row) {
    const int b = static_cast<int>(row / num_q_heads);
    const int h = static_cast<int>(row % num_q_heads);
    const int g = h / G;
    const int64_t L = seq_lens[b] > 0 ? seq_lens[b] : 0;
    const uint16_t* q_row = q + row * head_dim;
    const int32_t* table_row = block_table + static_cast<int64_t>(b) * block_table_stride;
    // sliding window: only the last `window` tokens are attended (window <= 0: all of them)
    const int64_t lo = (window > 0 && L > window) ? L - window : 0;
    if (chunk_tokens == 0) {
      attend_range(q_row, K, V, table_row, page_size, head_dim, g, sc, lo, L,
                   out + row * head_dim, lse + row);
    } else {
      const int64_t n_chunks = (L + chunk_tokens - 1) / chunk_tokens;
      for (int64_t c = 0; c < n_chunks; ++c) {
        int64_t t0 = c * chunk_tokens;
        const int64_t t1 = (t0 + chunk_tokens < L) ? t0 + chunk_tokens : L;
        if (t0 < lo) t0 = lo;  // a chunk wholly before the window is an empty range (o = 0, lse = -inf)
        attend_range(q_row, K, V, table_row, page_size, head_dim, g, sc, t0, t1,
                     out + (row * max_chunks + c) * head_dim, lse + row * max_chunks + c);
      }
    }
  });
}

// Append of n_new tokens per sequence: token i of new[b] (rows [B, n_new, Hkv, D])
// becomes logical token L_b - n_new + i, bytewise.
void oracle_kv_append_tokens(const uint8_t* k_new, const uint8_t* v_new, uint8_t* k_cache,
                             uint8_t* v_cache, int64_t page_stride, int64_t head_stride,
                             int64_t slot_stride, int32_t page_size, int32_t num_kv_heads,
                             int32_t head_dim, int32_t elem_bytes, const int32_t* block_table,
                             int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                             int32_t n_new) {
  for (int b = 0; b < batch; ++b) {
    const int64_t L = seq_lens[b];
    for (int i = 0; i < n_new; ++i) {
      const int64_t pos = L - n_new + i;
      if (L <= 0 || pos < 0) continue;
      const int64_t page = block_table[static_cast<int64_t>(b) * block_table_stride + pos / page_size];
      const int64_t slot = pos % page_size;
      for (int g = 0; g < num_kv_heads; ++g) {
        const int64_t dst = (page * page_stride + g * head_stride + slot * slot_stride) * elem_bytes;
        const int64_t src = ((static_cast<int64_t>(b) * n_new + i) * num_kv_heads + g) * head_dim * elem_bytes;
        std::memcpy(k_cache + dst, k_new + src, static_cast<size_t>(head_dim) * elem_bytes);
        std::memcpy(v_cache + dst, v_new + src, static_cast<size_t>(head_dim) * elem_bytes);
      }
    }
  }
}

// Quantising append into an e4m3 cache (one token per sequence; not in the paper,
// whose only remark on KV quantisation is that it did not help on its laptop
// scenario -- this is the policy of this library): for K and V separately and for
// every kv head, with x = the new bf16 row and slot = (L-1) % P of page
// block_table[b][(L-1)/P]:
//   slot == 0 (the page's first token): scale[page,g] = amax(x) * 2 / 448
//                                       (1 when amax == 0), stored;
//   slot  > 0: scale[page,g] is the value stored when the page was opened;
//   bytes = e4m3 nearest to x / scale (fp32 division, ties to the even code),
//           saturating at +-448 (later rows may exceed the first row's range).
// One row of the quantising append: the new bf16 row `src` becomes logical token `pos` of sequence b.
static void append_row_e4m3(const uint16_t* src, uint8_t* cache, float* scales, int64_t page_stride,
                            int64_t head_stride, int64_t slot_stride, int32_t page_size,
                            int32_t num_kv_heads, int32_t head_dim, const int32_t* table_row,
                            int64_t pos, int g, const double* pos_code) {
  const int64_t page = table_row[pos / page_size];
  const int64_t slot = pos % page_size;
  float& sc = scales[page * num_kv_heads + g];
  if (slot == 0) {
    float amax = 0.0f;
    for (int d = 0; d < head_dim; ++d) {
      const float a = std::fabs(static_cast<float>(bf16_to_double(src[d])));
      if (a > amax) amax = a;
    }
    sc = amax > 0.0f ? (amax * 2.0f) / 448.0f : 1.0f;
  }
  uint8_t* dst = cache + page * page_stride + g * head_stride + slot * slot_stride;
  for (int d = 0; d < head_dim; ++d) {
    const float y = static_cast<float>(bf16_to_double(src[d])) / sc;
    const double a = std::fabs(static_cast<double>(y));
    int best = 0;
    for (int i = 1; i < 127; ++i) {
      const double di = std::fabs(pos_code[i] - a), db = std::fabs(pos_code[best] - a);
      if (di < db || (di == db && (i % 2 == 0))) best = i;
    }
    dst[d] = static_cast<uint8_t>(best | (std::signbit(y) ? 0x80 : 0));
  }
}

void oracle_kv_append_e4m3(const uint16_t* k_new, const uint16_t* v_new, uint8_t* k_cache,
                           uint8_t* v_cache, float* k_scale, float* v_scale, int64_t page_stride,
                           int64_t head_stride, int64_t slot_stride, int32_t page_size,
                           int32_t num_kv_heads, int32_t head_dim, const int32_t* block_table,
                           int32_t block_table_stride, const int32_t* seq_lens, int32_t batch) {
  double pos[127];
  for (int i = 0; i < 127; ++i) pos[i] = e4m3_to_double(static_cast<uint8_t>(i));
  for (int b = 0; b < batch; ++b) {
    const int64_t L = seq_lens[b];
    if (L <= 0) continue;
    const int32_t* row = block_table + static_cast<int64_t>(b) * block_table_stride;
    for (int g = 0; g < num_kv_heads; ++g) {
      const int64_t src = (static_cast<int64_t>(b) * num_kv_heads + g) * head_dim;
      append_row_e4m3(k_new + src, k_cache, k_scale, page_stride, head_stride, slot_stride, page_size,
                      num_kv_heads, head_dim, row, L - 1, g, pos);
      append_row_e4m3(v_new + src, v_cache, v_scale, page_stride, head_stride, slot_stride, page_size,
                      num_kv_heads, head_dim, row, L - 1, g, pos);
    }
  }
}

// Quantising append of n_new tokens per sequence (rows [B, n_new, Hkv, D]): the one-token rule above
// applied to token i = 0, 1, ... in this order, token i standing at position L_b - n_new + i -- so a
// page opened inside the block takes its scale from the block's own row that lands in its slot 0.
void oracle_kv_append_tokens_e4m3(const uint16_t* k_new, const uint16_t* v_new, uint8_t* k_cache,
                                  uint8_t* v_cache, float* k_scale, float* v_scale,
                                  int64_t page_stride, int64_t head_stride, int64_t slot_stride,
                                  int32_t page_size, int32_t num_kv_heads, int32_t head_dim,
                                  const int32_t* block_table, int32_t block_table_stride,
                                  const int32_t* seq_lens, int32_t batch, int32_t n_new) {
  double pos[127];
  for (int i = 0; i < 127; ++i) pos[i] = e4m3_to_double(static_cast<uint8_t>(i));
  for (int b = 0; b < batch; ++b) {
    const int64_t L = seq_lens[b];
    if (L <= 0) continue;
    const int32_t* row = block_table + static_cast<int64_t>(b) * block_table_stride;
    for (int i = 0; i < n_new; ++i) {
      const int64_t at = L - n_new + i;
      if (at < 0) continue;
      for (int g = 0; g < num_kv_heads; ++g) {
        const int64_t src = ((static_cast<int64_t>(b) * n_new + i) * num_kv_heads + g) * head_dim;
        append_row_e4m3(k_new + src, k_cache, k_scale, page_stride, head_stride, slot_stride, page_size,
                        num_kv_heads, head_dim, row, at, g, pos);
        append_row_e4m3(v_new + src, v_cache, v_scale, page_stride, head_stride, slot_stride, page_size,
                        num_kv_heads, head_dim, row, at, g, pos);
      }
    }
  }
}

// Verification attention for a block of n_q query tokens per sequence (the
// predicted-output verifier of the paper's Scenario B scores a 16-token block
// in one pass; the paper gives no formula -- this is causal attention written
// out): the cache already holds all L_b tokens, the block being its last n_q;
// query token i stands at position L_b - n_q + i and attends tokens
// j <= L_b - n_q + i. q and out are [B, n_q, Hq, D], lse is [B, n_q, Hq].
void oracle_paged_verify_attention(
    const uint16_t* q, const uint8_t* k_cache, const uint8_t* v_cache, int32_t kv_dtype,
    const float* k_scale, const float* v_scale, int64_t page_stride, int64_t head_stride,
    int64_t slot_stride, int32_t page_size, int32_t num_kv_heads, int32_t head_dim,
    const int32_t* block_table, int32_t block_table_stride, const int32_t* seq_lens,
    int32_t batch, int32_t num_q_heads, int32_t n_q, float scale, double* out, double* lse,
    int32_t n_threads) {
  const int G = num_q_heads / num_kv_heads;
  const CacheView K{k_cache, kv_dtype, page_stride, head_stride, slot_stride, k_scale, num_kv_heads};
  const CacheView V{v_cache, kv_dtype, page_stride, head_stride, slot_stride, v_scale, num_kv_heads};
  const double sc = static_cast<double>(scale);
  const int64_t rows = static_cast<int64_t>(batch) * n_q * num_q_heads;
  parallel_for(rows, n_threads, [&](int64_t row) {
    const int h = static_cast<int>(row % num_q_heads);
    const int i = static_cast<int>((row / num_q_heads) % n_q);
    const int b = static_cast<int>(row / (static_cast<int64_t>(num_q_heads) * n_q));
    const int64_t L = seq_lens[b] > 0 ? seq_lens[b] : 0;
    int64_t limit = L - n_q + i + 1;  // number of visible tokens
    if (limit < 0) limit = 0;
    if (limit > L) limit = L;
    attend_range(q + row * head_dim, K, V, block_table + static_cast<int64_t>(b) * block_table_stride,
                 page_size, head_dim, h / G, sc, 0, limit, out + row * head_dim, lse + row);
  });
}

// Merge of split-KV partials: each chunk's o_c is already normalised within the
// chunk and lse_c = m_c + log(l_c), so the full softmax average is
//   out = sum_c w_c o_c / sum_c w_c,  w_c = exp(lse_c - max_c lse_c).
// n_chunks(b) = ceil(L_b / chunk_tokens); a sequence with no chunk gives 0.
void oracle_paged_decode_reduce(const double* part_o, const double* part_lse,
                                const int32_t* seq_lens, int32_t batch, int32_t num_q_heads,
                                int32_t head_dim, int32_t chunk_tokens, int32_t max_chunks,
                                double* out, double* lse) {
  for (int64_t row = 0; row < static_cast<int64_t>(batch) * num_q_heads; ++row) {
    const int b = static_cast<int>(row / num_q_heads);
    const int64_t L = seq_lens[b] > 0 ? seq_lens[b] : 0;
    const int64_t n_chunks = (L + chunk_tokens - 1) / chunk_tokens;
    double* o = out + row * head_dim;
    for (int d = 0; d < head_dim; ++d) o[d] = 0.0;
    double M = -std::numeric_limits<double>::infinity();
    for (int64_t c = 0; c < n_chunks; ++c) {
      const double v = part_lse[row * max_chunks + c];
      if (v > M) M = v;
    }
    if (n_chunks == 0 || !(M > -std::numeric_limits<double>::infinity())) {
      if (lse) lse[row] = -std::numeric_limits<double>::infinity();
      continue;
    }
    double W = 0.0;
    for (int64_t c = 0; c < n_chunks; ++c) {
      const double w = std::exp(part_lse[row * max_chunks + c] - M);
      W += w;
      const double* oc = part_o + (row * max_chunks + c) * head_dim;
      for (int d = 0; d < head_dim; ++d) o[d] += w * oc[d];
    }
    for (int d = 0; d < head_dim; ++d) o[d] /= W;
    if (lse) lse[row] = M + std::log(W);
  }
}

// Input preparation for e4m3 caches: for each (page, kv head) tile of a bf16
// cache laid out [num_pages, Hkv, P, D] contiguously, scale = amax / 448 over
// the first valid_slots[page] slots (scale = 1 when amax == 0), and every
// element of those slots becomes the e4m3 value nearest to x / scale
// (fp32 division, round to nearest, ties to the even code, saturating at
// +-448). Slots at or beyond valid_slots[page] keep the bytes already in dst.
void oracle_quantize_pages_e4m3(const uint16_t* src, const int32_t* valid_slots,
                                int32_t num_pages, int32_t num_kv_heads, int32_t page_size,
                                int32_t head_dim, uint8_t* dst, float* scales) {
  double pos[127];  // codes 0x00..0x7E, increasing
  for (int i = 0; i < 127; ++i) pos[i] = e4m3_to_double(static_cast<uint8_t>(i));
  for (int64_t page = 0; page < num_pages; ++page) {
    const int valid = valid_slots[page];
    for (int g = 0; g < num_kv_heads; ++g) {
      const int64_t tile = (page * num_kv_heads + g) * page_size * head_dim;
      float amax = 0.0f;
      for (int s = 0; s < valid; ++s)
        for (int d = 0; d < head_dim; ++d) {
          const float a = std::fabs(static_cast<float>(bf16_to_double(src[tile + s * head_dim + d])));
          if (a > amax) amax = a;
        }
      const float sc = amax > 0.0f ? amax / 448.0f : 1.0f;
      scales[page * num_kv_heads + g] = sc;
      for (int s = 0; s < valid; ++s)
        for (int d = 0; d < head_dim; ++d) {
          const float x = static_cast<float>(bf16_to_double(src[tile + s * head_dim + d]));
          const float y = x / sc;
          const double a = std::fabs(static_cast<double>(y));
          int best = 0;
          for (int i = 1; i < 127; ++i) {
            const double di = std::fabs(pos[i] - a), db = std::fabs(pos[best] - a);
            if (di < db || (di == db && (i % 2 == 0))) best = i;
          }
          dst[tile + s * head_dim + d] = static_cast<uint8_t>(best | (std::signbit(y) ? 0x80 : 0));
        }
    }
  }
}

}  // extern "C"
