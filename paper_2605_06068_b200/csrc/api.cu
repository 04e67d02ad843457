// C ABI of libpda: argument validation on the host, then kernel dispatch.
#include <atomic>
#include <cstdint>
#include <mutex>

#include "common.cuh"

namespace {

using pda::AttnParams;
using pda::CacheGeom;

// units per resident CTA from which paged_decode_step uses the persistent kernel (unsplit launches)
std::atomic<int> g_persist_min_units{6};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks the cache descriptor; on success fills `g`.
int check_desc(const pda_cache_desc* d, CacheGeom* g) {
  if (d == nullptr) return PDA_ERR_INVALID_ARG;
  if (d->num_pages < 0 || d->num_kv_heads <= 0 || d->head_dim <= 0 || d->page_size <= 0)
    return PDA_ERR_INVALID_ARG;
  if (d->dtype != PDA_BF16 && d->dtype != PDA_FP8_E4M3) return PDA_ERR_UNSUPPORTED;
  if (d->page_size != pda::kPageSize) return PDA_ERR_UNSUPPORTED;
  if (d->head_dim % 32 != 0 || d->head_dim > 256) return PDA_ERR_UNSUPPORTED;
  if (d->page_stride <= 0 || d->head_stride <= 0 || d->slot_stride < d->head_dim)
    return PDA_ERR_INVALID_ARG;
  const int64_t eb = d->dtype == PDA_BF16 ? 2 : 1;
  if ((d->page_stride * eb) % 16 || (d->head_stride * eb) % 16 || (d->slot_stride * eb) % 16)
    return PDA_ERR_MISALIGNED;
  g->page_stride = d->page_stride;
  g->head_stride = d->head_stride;
  g->slot_stride = d->slot_stride;
  g->num_pages = d->num_pages;
  g->num_kv_heads = d->num_kv_heads;
  g->head_dim = d->head_dim;
  g->dtype = d->dtype;
  return PDA_OK;
}

int check_attention(const void* q, const void* k_cache, const void* v_cache,
                    const pda_cache_desc* desc, const float* k_scale, const float* v_scale,
                    const int32_t* block_table, int32_t block_table_stride,
                    const int32_t* seq_lens, int32_t batch, int32_t num_q_heads,
                    int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                    int32_t max_chunks, AttnParams* p) {
  CacheGeom g;
  if (int rc = check_desc(desc, &g)) return rc;
  if (batch < 0 || num_q_heads <= 0 || block_table_stride < 0 || chunk_tokens < 0)
    return PDA_ERR_INVALID_ARG;
  if (num_q_heads % g.num_kv_heads != 0) return PDA_ERR_INVALID_ARG;
  if (chunk_tokens % pda::kPageSize != 0) return PDA_ERR_INVALID_ARG;
  if (batch > 65535 || num_q_heads > 65535) return PDA_ERR_TOO_LARGE;
  if (batch > 0) {
    if (!q || !k_cache || !v_cache || !block_table || !seq_lens) return PDA_ERR_INVALID_ARG;
    if (block_table_stride == 0) return PDA_ERR_INVALID_ARG;
    if (g.dtype == PDA_FP8_E4M3 && (!k_scale || !v_scale)) return PDA_ERR_INVALID_ARG;
    if (chunk_tokens == 0) {
      if (!out) return PDA_ERR_INVALID_ARG;
    } else {
      if (!part_o || !part_lse || max_chunks <= 0) return PDA_ERR_INVALID_ARG;
    }
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) ||
        (chunk_tokens == 0 && !aligned16(out)) || (chunk_tokens > 0 && !aligned16(part_o)))
      return PDA_ERR_MISALIGNED;
  }
  p->q = static_cast<const __nv_bfloat16*>(q);
  p->k_cache = k_cache;
  p->v_cache = v_cache;
  p->k_scale = k_scale;
  p->v_scale = v_scale;
  p->block_table = block_table;
  p->seq_lens = seq_lens;
  p->out = static_cast<__nv_bfloat16*>(out);
  p->part_o = part_o;
  p->part_lse = part_lse;
  p->status = nullptr;
  p->geom = g;
  p->block_table_stride = block_table_stride;
  p->batch = batch;
  p->num_q_heads = num_q_heads;
  p->group = num_q_heads / g.num_kv_heads;
  p->chunk_tokens = chunk_tokens;
  p->max_chunks = max_chunks;
  p->scale = 0.f;
  p->window = 0;
  p->first_token = 0;
  p->chunk_slot0 = 0;
  return PDA_OK;
}

}  // namespace

namespace {
// A library-owned second stream for the one place where two independent launches of a call can share
// the GPU (the shared-prefix cascade: its prefix launch leaves SMs idle that the suffix launch can use).
// Fork and join go through events, so the pattern is also valid inside a stream capture. One set per
// device, created by the first call on that device that is not being captured (creating a stream during
// a capture is not allowed in every capture mode); until then such calls run their launches one after
// the other, as they do on a device beyond kMaxDevices.
struct SideStream {
  std::mutex mu;
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
constexpr int kMaxDevices = 64;
SideStream g_side[kMaxDevices];

// The current device's set, or nullptr when there is none to use.
SideStream* side_stream_of_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return dev >= 0 && dev < kMaxDevices ? &g_side[dev] : nullptr;
}

bool side_stream_ready(SideStream& side, cudaStream_t main_stream) {  // side.mu held, side's device current
  if (side.stream) return true;
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(main_stream, &st) != cudaSuccess || st != cudaStreamCaptureStatusNone) {
    cudaGetLastError();
    return false;
  }
  cudaStream_t ns = nullptr;
  cudaEvent_t a = nullptr, b = nullptr;
  if (cudaStreamCreateWithFlags(&ns, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
    cudaGetLastError();
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (ns) cudaStreamDestroy(ns);
    return false;
  }
  side.stream = ns;
  side.fork = a;
  side.join = b;
  return true;
}

// Device address of pinned, mapped host memory (what cudaHostAlloc / cudaHostRegister give); NULL for
// anything the device cannot reach.
void* mapped_device_pointer(const void* host) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  if (a.type != cudaMemoryTypeHost && a.type != cudaMemoryTypeManaged && a.type != cudaMemoryTypeDevice)
    return nullptr;
  return a.devicePointer;
}
}  // namespace

extern "C" {

int pda_version(void) { return PDA_VERSION; }

const char* pda_status_string(int code) {
  switch (code) {
    case PDA_OK: return "ok";
    case PDA_ERR_INVALID_ARG: return "invalid argument";
    case PDA_ERR_UNSUPPORTED: return "unsupported shape, dtype or layout";
    case PDA_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case PDA_ERR_TOO_LARGE: return "size beyond a fixed maximum";
    case PDA_DEV_BAD_PAGE: return "device: block_table entry out of range";
    case PDA_DEV_BAD_SEQ_LEN: return "device: seq_len exceeds block_table capacity";
    case PDA_DEV_TIMEOUT: return "device: bounded wait on an asynchronous copy expired";
    default: return code > 0 ? "cuda error or unknown device status" : "unknown error";
  }
}

int pda_max_chunks(int32_t max_seq_len, int32_t chunk_tokens) {
  if (chunk_tokens <= 0 || max_seq_len < 0) return PDA_ERR_INVALID_ARG;
  return static_cast<int>((static_cast<int64_t>(max_seq_len) + chunk_tokens - 1) / chunk_tokens);
}

int kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
              const pda_cache_desc* desc, const int32_t* block_table,
              int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
              int32_t* status, pda_stream_t stream) {
  CacheGeom g;
  if (int rc = check_desc(desc, &g)) return rc;
  if (g.dtype != PDA_BF16) return PDA_ERR_UNSUPPORTED;
  if (batch < 0 || block_table_stride < 0) return PDA_ERR_INVALID_ARG;
  if (batch == 0) return PDA_OK;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !seq_lens ||
      block_table_stride == 0)
    return PDA_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache))
    return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_kv_append(k_new, v_new, k_cache, v_cache, g, block_table,
                                                block_table_stride, seq_lens, batch, status,
                                                static_cast<cudaStream_t>(stream)));
}

int paged_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                           const pda_cache_desc* desc, const float* k_scale,
                           const float* v_scale, const int32_t* block_table,
                           int32_t block_table_stride, const int32_t* seq_lens,
                           int32_t batch, int32_t num_q_heads, float scale,
                           int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                           int32_t max_chunks, uint32_t flags, int32_t* status,
                           pda_stream_t stream) {
  AttnParams p;
  if (int rc = check_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                               block_table_stride, seq_lens, batch, num_q_heads, chunk_tokens,
                               out, part_o, part_lse, max_chunks, &p))
    return rc;
  if (batch == 0) return PDA_OK;
  p.status = status;
  p.scale = scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!(flags & PDA_FLAG_FORCE_GENERIC) && pda::attention_tma_supports(p))
    return static_cast<int>(pda::launch_attention_tma(p, s));
  return static_cast<int>(pda::launch_attention_generic(p, s));
}

int paged_window_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                                  const pda_cache_desc* desc, const float* k_scale,
                                  const float* v_scale, const int32_t* block_table,
                                  int32_t block_table_stride, const int32_t* seq_lens,
                                  int32_t batch, int32_t num_q_heads, float scale, int32_t window,
                                  int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                                  int32_t max_chunks, uint32_t flags, int32_t* status,
                                  pda_stream_t stream) {
  AttnParams p;
  if (window < 0) return PDA_ERR_INVALID_ARG;
  if (int rc = check_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                               block_table_stride, seq_lens, batch, num_q_heads, chunk_tokens,
                               out, part_o, part_lse, max_chunks, &p))
    return rc;
  if (batch == 0) return PDA_OK;
  p.status = status;
  p.scale = scale;
  p.window = window;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!(flags & PDA_FLAG_FORCE_GENERIC) && pda::attention_tma_supports(p))
    return static_cast<int>(pda::launch_attention_tma(p, s));
  return static_cast<int>(pda::launch_attention_generic(p, s));
}

int kv_append_tokens(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                     const pda_cache_desc* desc, const int32_t* block_table,
                     int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                     int32_t n_new, int32_t* status, pda_stream_t stream) {
  CacheGeom g;
  if (int rc = check_desc(desc, &g)) return rc;
  if (g.dtype != PDA_BF16) return PDA_ERR_UNSUPPORTED;
  if (batch < 0 || block_table_stride < 0 || n_new < 0) return PDA_ERR_INVALID_ARG;
  if (batch == 0 || n_new == 0) return PDA_OK;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !seq_lens ||
      block_table_stride == 0)
    return PDA_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache))
    return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_kv_append_tokens(k_new, v_new, k_cache, v_cache, g,
                                                       block_table, block_table_stride, seq_lens,
                                                       batch, n_new, status,
                                                       static_cast<cudaStream_t>(stream)));
}

namespace {
int append_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
               const pda_cache_desc* desc, float* k_scale, float* v_scale, const int32_t* block_table,
               int32_t block_table_stride, const int32_t* seq_lens, int32_t batch, int32_t n_new,
               int32_t* status, pda_stream_t stream) {
  CacheGeom g;
  if (int rc = check_desc(desc, &g)) return rc;
  if (g.dtype != PDA_FP8_E4M3 || g.head_dim % 64 != 0) return PDA_ERR_UNSUPPORTED;
  if (batch < 0 || block_table_stride < 0 || n_new < 0) return PDA_ERR_INVALID_ARG;
  if (batch == 0 || n_new == 0) return PDA_OK;
  if (!k_new || !v_new || !k_cache || !v_cache || !k_scale || !v_scale || !block_table ||
      !seq_lens || block_table_stride == 0)
    return PDA_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache))
    return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_kv_append_e4m3(k_new, v_new, k_cache, v_cache, k_scale,
                                                     v_scale, g, block_table, block_table_stride,
                                                     seq_lens, batch, n_new, status,
                                                     static_cast<cudaStream_t>(stream)));
}
}  // namespace

int kv_append_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  const pda_cache_desc* desc, float* k_scale, float* v_scale,
                  const int32_t* block_table, int32_t block_table_stride,
                  const int32_t* seq_lens, int32_t batch, int32_t* status, pda_stream_t stream) {
  return append_fp8(k_new, v_new, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                    block_table_stride, seq_lens, batch, 1, status, stream);
}

int kv_append_tokens_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         const pda_cache_desc* desc, float* k_scale, float* v_scale,
                         const int32_t* block_table, int32_t block_table_stride,
                         const int32_t* seq_lens, int32_t batch, int32_t n_new, int32_t* status,
                         pda_stream_t stream) {
  return append_fp8(k_new, v_new, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                    block_table_stride, seq_lens, batch, n_new, status, stream);
}

int paged_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                           const pda_cache_desc* desc, const float* k_scale,
                           const float* v_scale, const int32_t* block_table,
                           int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                           int32_t num_q_heads, int32_t n_query_tokens, float scale,
                           int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                           int32_t max_chunks, uint32_t flags, int32_t* status,
                           pda_stream_t stream) {
  AttnParams p;
  if (n_query_tokens <= 0 || n_query_tokens > 4096) return PDA_ERR_INVALID_ARG;
  if (!out && batch > 0) return PDA_ERR_INVALID_ARG;
  if (int rc = check_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                               block_table_stride, seq_lens, batch, num_q_heads, chunk_tokens,
                               out, part_o, part_lse, max_chunks, &p))
    return rc;
  if (static_cast<int64_t>(batch) * n_query_tokens > 65535) return PDA_ERR_TOO_LARGE;
  if (batch == 0) return PDA_OK;
  p.status = status;
  p.scale = scale;
  p.out = static_cast<__nv_bfloat16*>(out);
  pda::MqParams mp{p, n_query_tokens, 1, 0, max_chunks};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!(flags & (PDA_FLAG_MQ_MMA_SYNC | PDA_FLAG_MQ_ONE_UNIT)) && pda::attention_mq_tcp_supports(mp)) {
    if (cudaError_t e = pda::launch_attention_mq_tcp(mp, s)) return static_cast<int>(e);
  } else if (!(flags & (PDA_FLAG_MQ_MMA_SYNC | PDA_FLAG_MQ_ONE_UNIT)) && pda::attention_mq_tc8p_supports(mp)) {
    if (cudaError_t e = pda::launch_attention_mq_tc8p(mp, s)) return static_cast<int>(e);
  } else if (!(flags & PDA_FLAG_MQ_MMA_SYNC) && pda::attention_mq_tc_supports(mp)) {
    if (cudaError_t e = pda::launch_attention_mq_tc(mp, s)) return static_cast<int>(e);
  } else {
    if (!pda::attention_mq_supports(mp)) return PDA_ERR_UNSUPPORTED;
    if (cudaError_t e = pda::launch_attention_mq(mp, s)) return static_cast<int>(e);
  }
  if (chunk_tokens > 0)
    return static_cast<int>(pda::launch_reduce(part_o, part_lse, seq_lens, batch, num_q_heads,
                                               p.geom.head_dim, chunk_tokens, max_chunks, 0, 0,
                                               n_query_tokens, static_cast<__nv_bfloat16*>(out), s));
  return PDA_OK;
}

int paged_prefix_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                                  const pda_cache_desc* desc, const float* k_scale,
                                  const float* v_scale, const int32_t* block_table,
                                  int32_t block_table_stride, const int32_t* seq_lens,
                                  int32_t batch, int32_t num_q_heads, float scale,
                                  int32_t prefix_tokens, int32_t prefix_chunk_tokens,
                                  int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                                  int32_t max_chunks, uint32_t flags, int32_t* status,
                                  pda_stream_t stream) {
  AttnParams p;
  if (prefix_tokens <= 0 || prefix_chunk_tokens <= 0 || chunk_tokens <= 0) return PDA_ERR_INVALID_ARG;
  if (prefix_tokens % pda::kPageSize || prefix_chunk_tokens % pda::kPageSize) return PDA_ERR_INVALID_ARG;
  if (!out && batch > 0) return PDA_ERR_INVALID_ARG;
  if (int rc = check_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                               block_table_stride, seq_lens, batch, num_q_heads, chunk_tokens,
                               out, part_o, part_lse, max_chunks, &p))
    return rc;
  const int prefix_chunks = (prefix_tokens + prefix_chunk_tokens - 1) / prefix_chunk_tokens;
  if (prefix_chunks >= max_chunks) return PDA_ERR_INVALID_ARG;
  if (static_cast<int64_t>(prefix_tokens) > static_cast<int64_t>(block_table_stride) * pda::kPageSize)
    return PDA_ERR_INVALID_ARG;
  if (batch == 0) return PDA_OK;
  p.status = status;
  p.scale = scale;
  p.out = static_cast<__nv_bfloat16*>(out);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // (1) the shared prefix once: the batch's queries as one block of rows per kv head
  AttnParams pp = p;
  pp.batch = 1;
  pp.chunk_tokens = prefix_chunk_tokens;
  pp.chunk_slot0 = 0;
  pda::MqParams mp{pp, batch, 0, prefix_tokens, prefix_chunks};
  const bool prefix_tc = !(flags & PDA_FLAG_MQ_MMA_SYNC) && pda::attention_mq_tc_supports(mp);
  if (!pda::attention_tma_supports(p) || (!prefix_tc && !pda::attention_mq_supports(mp)))
    return PDA_ERR_UNSUPPORTED;  // (decided before anything is enqueued)

  // The suffix launch (2) is independent of the prefix launch (1) and small, and (1) rarely fills the
  // GPU (one CTA per SM, chunks x kv heads of them), so (2) runs beside it on the library's second
  // stream: the fork event is recorded before (1), (1) is submitted first so that its CTAs are placed
  // first, and (2) is joined before the merge.
  static std::mutex no_side_mu;  // (a device without a set: nothing to guard, the launches stay on `stream`)
  SideStream* side = side_stream_of_current_device();
  std::lock_guard<std::mutex> lock(side ? side->mu : no_side_mu);
  bool forked = side && side_stream_ready(*side, s) && cudaEventRecord(side->fork, s) == cudaSuccess;
  if (!forked) cudaGetLastError();

  if (cudaError_t e = prefix_tc ? pda::launch_attention_mq_tc(mp, s) : pda::launch_attention_mq(mp, s))
    return static_cast<int>(e);
  // (2) every sequence's own suffix, chunk slots after the prefix's
  AttnParams ps = p;
  ps.first_token = prefix_tokens;
  ps.chunk_slot0 = prefix_chunks;
  if (forked && cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess) {
    cudaGetLastError();
    forked = false;
  }
  cudaError_t e2 = pda::launch_attention_tma(ps, forked ? side->stream : s);
  if (forked) {  // join in any case: a capture must not be left with an open branch
    cudaError_t ej = cudaEventRecord(side->join, side->stream);
    if (ej == cudaSuccess) ej = cudaStreamWaitEvent(s, side->join, 0);
    if (e2 == cudaSuccess) e2 = ej;
  }
  if (e2 != cudaSuccess) return static_cast<int>(e2);
  // (3) merge
  return static_cast<int>(pda::launch_reduce(part_o, part_lse, seq_lens, batch, num_q_heads,
                                             p.geom.head_dim, chunk_tokens, max_chunks,
                                             prefix_tokens, prefix_chunks, 1,
                                             static_cast<__nv_bfloat16*>(out), s));
}

int pda_set_persistent_threshold(int32_t min_units_per_cta) {
  if (min_units_per_cta < 0) return PDA_ERR_INVALID_ARG;
  g_persist_min_units.store(min_units_per_cta);
  return PDA_OK;
}

int pda_workspace_ints(int32_t batch, int32_t num_kv_heads) {
  if (batch < 0 || num_kv_heads <= 0) return PDA_ERR_INVALID_ARG;
  const int64_t n = 2 + static_cast<int64_t>(batch) * num_kv_heads;
  return n > INT32_MAX ? PDA_ERR_TOO_LARGE : static_cast<int>(n);
}

int paged_decode_step(const void* q, const void* k_new, const void* v_new, void* k_cache,
                      void* v_cache, const pda_cache_desc* desc, const float* k_scale,
                      const float* v_scale, const int32_t* block_table,
                      int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                      int32_t num_q_heads, float scale, int32_t chunk_tokens, void* out,
                      float* part_o, float* part_lse, int32_t max_chunks, int32_t* workspace,
                      int32_t* status, pda_stream_t stream) {
  AttnParams p;
  if (!out && batch > 0) return PDA_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return PDA_ERR_INVALID_ARG;
  if (int rc = check_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                               block_table_stride, seq_lens, batch, num_q_heads, chunk_tokens,
                               out, part_o, part_lse, max_chunks, &p))
    return rc;
  if (k_new && p.geom.dtype != PDA_BF16) return PDA_ERR_UNSUPPORTED;
  if (k_new && (!aligned16(k_new) || !aligned16(v_new))) return PDA_ERR_MISALIGNED;
  if (batch == 0) return PDA_OK;
  p.status = status;
  p.scale = scale;
  p.out = static_cast<__nv_bfloat16*>(out);
  const bool can_fuse = pda::attention_tma_supports(p) && (chunk_tokens == 0 || workspace);
  if (can_fuse) {
    pda::StepParams sp{p, k_new, v_new, k_cache, v_cache, workspace, 1};
    if (pda::attention_persist_supports(sp) && pda::attention_persist_preferred(sp, g_persist_min_units))
      return static_cast<int>(pda::launch_attention_persist(sp, static_cast<cudaStream_t>(stream)));
    return static_cast<int>(pda::launch_step_tma(sp, static_cast<cudaStream_t>(stream)));
  }
  // shapes outside the fused kernel: the same step as separate launches
  if (k_new) {
    if (int rc = kv_append(k_new, v_new, k_cache, v_cache, desc, block_table, block_table_stride,
                           seq_lens, batch, status, stream))
      return rc;
  }
  if (int rc = paged_decode_attention(q, k_cache, v_cache, desc, k_scale, v_scale, block_table,
                                      block_table_stride, seq_lens, batch, num_q_heads, scale,
                                      chunk_tokens, out, part_o, part_lse, max_chunks, 0u, status,
                                      stream))
    return rc;
  if (chunk_tokens > 0)
    return paged_decode_reduce(part_o, part_lse, seq_lens, batch, num_q_heads, p.geom.head_dim,
                               chunk_tokens, max_chunks, out, stream);
  return PDA_OK;
}

int paged_decode_reduce(const float* part_o, const float* part_lse, const int32_t* seq_lens,
                        int32_t batch, int32_t num_q_heads, int32_t head_dim,
                        int32_t chunk_tokens, int32_t max_chunks, void* out,
                        pda_stream_t stream) {
  if (batch < 0 || num_q_heads <= 0 || head_dim <= 0 || chunk_tokens <= 0 || max_chunks <= 0)
    return PDA_ERR_INVALID_ARG;
  if (batch > 65535 || num_q_heads > 65535) return PDA_ERR_TOO_LARGE;
  if (batch == 0) return PDA_OK;
  if (!part_o || !part_lse || !seq_lens || !out) return PDA_ERR_INVALID_ARG;
  if (head_dim % 4 != 0) return PDA_ERR_UNSUPPORTED;
  if (!aligned16(part_o) || (reinterpret_cast<uintptr_t>(out) & 7u)) return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_reduce(part_o, part_lse, seq_lens, batch, num_q_heads,
                                             head_dim, chunk_tokens, max_chunks, 0, 0, 1,
                                             static_cast<__nv_bfloat16*>(out),
                                             static_cast<cudaStream_t>(stream)));
}

int paged_decode_step_host(const void* q_host, const void* k_new_host, const void* v_new_host,
                           const int32_t* block_table_host, const int32_t* seq_lens_host,
                           void* q_dev, void* k_new_dev, void* v_new_dev,
                           int32_t* block_table_dev, int32_t* seq_lens_dev,
                           void* k_cache, void* v_cache, const pda_cache_desc* desc,
                           int32_t block_table_stride, int32_t batch, int32_t num_q_heads,
                           float scale, int32_t chunk_tokens, float* part_o, float* part_lse,
                           int32_t max_chunks, int32_t* workspace, void* out_dev, void* out_host,
                           int32_t* status, pda_stream_t stream) {
  AttnParams p;
  if (!out_host || !q_host || !k_new_host || !v_new_host) return PDA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // A staging buffer that is NULL means "in place": the kernel reads (writes) the host buffer itself
  // over the bus, which needs pinned, device-mapped host memory.
  const void* q_use = q_dev;
  const void* k_use = k_new_dev;
  const void* v_use = v_new_dev;
  void* out_use = out_dev;
  const int32_t* bt_use = block_table_dev;
  const int32_t* sl_use = seq_lens_dev;
  if (batch > 0 && (!block_table_host || !seq_lens_host)) return PDA_ERR_INVALID_ARG;
  if (!q_dev && !(q_use = mapped_device_pointer(q_host))) return PDA_ERR_INVALID_ARG;
  if (!k_new_dev && !(k_use = mapped_device_pointer(k_new_host))) return PDA_ERR_INVALID_ARG;
  if (!v_new_dev && !(v_use = mapped_device_pointer(v_new_host))) return PDA_ERR_INVALID_ARG;
  if (!out_dev && !(out_use = mapped_device_pointer(out_host))) return PDA_ERR_INVALID_ARG;
  if (batch > 0 && !block_table_dev &&
      !(bt_use = static_cast<const int32_t*>(mapped_device_pointer(block_table_host))))
    return PDA_ERR_INVALID_ARG;
  if (batch > 0 && !seq_lens_dev &&
      !(sl_use = static_cast<const int32_t*>(mapped_device_pointer(seq_lens_host))))
    return PDA_ERR_INVALID_ARG;
  if (int rc = check_attention(q_use, k_cache, v_cache, desc, nullptr, nullptr, bt_use,
                               block_table_stride, sl_use, batch, num_q_heads,
                               chunk_tokens, out_use, part_o, part_lse, max_chunks, &p))
    return rc;
  if (p.geom.dtype != PDA_BF16) return PDA_ERR_UNSUPPORTED;
  if (batch == 0) return PDA_OK;
  // The two copies every CTA depends on go first: as one small kernel that reads both host buffers over
  // the bus when they are mapped into the device's address space and nothing else of this step goes
  // through the copy engine (cheaper than two copy calls: 109 against 118 us per llama8b step), else as
  // two copies.
  cudaError_t e;
  const int32_t* bt_map = nullptr;
  const int32_t* sl_map = nullptr;
  const bool copies_anyway = q_dev || k_new_dev || v_new_dev;  // (mixing copy-engine work and a kernel only adds hand-overs)
  if (!copies_anyway && block_table_dev && seq_lens_dev &&
      (bt_map = static_cast<const int32_t*>(mapped_device_pointer(block_table_host))) != nullptr &&
      (sl_map = static_cast<const int32_t*>(mapped_device_pointer(seq_lens_host))) != nullptr) {
    if ((e = pda::launch_stage_tables(bt_map, block_table_dev, static_cast<int64_t>(batch) * block_table_stride,
                                      sl_map, seq_lens_dev, batch, s)))
      return e;
  } else {
    if (block_table_dev && (e = cudaMemcpyAsync(block_table_dev, block_table_host,
                                                static_cast<size_t>(batch) * block_table_stride * 4,
                                                cudaMemcpyHostToDevice, s)))
      return e;
    if (seq_lens_dev && (e = cudaMemcpyAsync(seq_lens_dev, seq_lens_host, static_cast<size_t>(batch) * 4,
                                             cudaMemcpyHostToDevice, s)))
      return e;
  }
  const size_t D = p.geom.head_dim;
  const size_t q_bytes = static_cast<size_t>(batch) * num_q_heads * D * 2;
  const size_t new_bytes = static_cast<size_t>(batch) * p.geom.num_kv_heads * D * 2;
  if (q_dev && (e = cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, s))) return e;
  if (k_new_dev && (e = cudaMemcpyAsync(k_new_dev, k_new_host, new_bytes, cudaMemcpyHostToDevice, s))) return e;
  if (v_new_dev && (e = cudaMemcpyAsync(v_new_dev, v_new_host, new_bytes, cudaMemcpyHostToDevice, s))) return e;
  if (int rc = paged_decode_step(q_use, k_use, v_use, k_cache, v_cache, desc, nullptr, nullptr,
                                 bt_use, block_table_stride, sl_use, batch,
                                 num_q_heads, scale, chunk_tokens, out_use, part_o, part_lse,
                                 max_chunks, workspace, status, stream))
    return rc;
  if (out_dev && (e = cudaMemcpyAsync(out_host, out_dev, q_bytes, cudaMemcpyDeviceToHost, s))) return e;
  return PDA_OK;
}

int pda_advance_seq_lens(int32_t* seq_lens, int32_t batch, int32_t delta, pda_stream_t stream) {
  if (batch < 0) return PDA_ERR_INVALID_ARG;
  if (batch == 0) return PDA_OK;
  if (!seq_lens) return PDA_ERR_INVALID_ARG;
  return static_cast<int>(pda::launch_advance_seq_lens(seq_lens, batch, delta,
                                                       static_cast<cudaStream_t>(stream)));
}

int pda_debug_e4m3_decode(float* out256, pda_stream_t stream) {
  if (!out256) return PDA_ERR_INVALID_ARG;
  return static_cast<int>(pda::launch_e4m3_decode(out256, static_cast<cudaStream_t>(stream)));
}

int pda_debug_wait_timeout(uint32_t polls, int32_t* status, uint64_t* result, pda_stream_t stream) {
  if (!status || polls == 0 || polls > (1u << 20)) return PDA_ERR_INVALID_ARG;
  if (result && (reinterpret_cast<uintptr_t>(result) & 7u)) return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_wait_timeout(polls, status, result, static_cast<cudaStream_t>(stream)));
}

int pda_debug_read_probe(const void* buf, uint64_t bytes, uint32_t* sink, pda_stream_t stream) {
  if (!buf || !sink || bytes == 0 || bytes % 16 != 0) return PDA_ERR_INVALID_ARG;
  if (!aligned16(buf)) return PDA_ERR_MISALIGNED;
  return static_cast<int>(pda::launch_read_probe(buf, static_cast<size_t>(bytes), sink,
                                                 static_cast<cudaStream_t>(stream)));
}

}  // extern "C"
