// Multi-query paged attention on the 5th-generation tensor cores (tcgen05 + TMEM): verification of a
// block of draft tokens, and the shared-prefix part of a decode batch; same contract as attention_mq.cu.
// Up to 128 query rows (query tokens x group size) per CTA against one sequence's pages. bf16 KV with
// head_dim 128 or 64 (the figures in this comment are for bf16 and 128), or e4m3 KV with head_dim 128.
//
// This is the part of the path that is a real dense contraction, so it runs as
// UMMA tiles with operands and accumulators in tensor memory (TMEM, 128 lanes = query rows):
//   S[128 x 64]  = Q[128 x D] . K^T     per 4 pages: 8 tcgen05.mma of M128 x N64 x K16
//                                        (A = Q in TMEM, B = K, K-major; the 4 pages' rows are stacked)
//   O[128 x D]  += P[128 x 64] . V      per page 1 tcgen05.mma M128 x N128 x K16
//                                        (A = P in TMEM, B = V, MN-major)
//   l[128]      += P[128 x 64] . 1      per page 1 tcgen05.mma M128 x N16 x K16 against a tile of ones:
//                                        the row sums of exactly the bf16 P that multiplies V
// Only K and V are read from shared memory by the tensor core (with A there too an N = 64 MMA is bound
// by shared-memory bandwidth: 50 instead of 33 clocks, measured). The (page, head) tiles land through
// the same 5-D TMA maps as everywhere else: rows of 128-byte lines with the 128-byte swizzle are already
// the canonical UMMA layouts, K-major for K (rows = tokens, contraction over d; copied line by line so
// that the 4 pages of an iteration stack to [line][64 tokens][128 B]) and MN-major for V (contraction
// over the 16 tokens of a page), so no data is rearranged in shared memory.
//
// Warp roles (11 warps): 0-3 and 4-7 two softmax sets (TMEM lane t <-> query row t; set x takes the
// iterations it with it % 2 == x, so each scheduler holds one warp of each set and one covers the
// other's waits), 8 TMA producer, 9 S issue + TMEM allocation, 10 PV issue (one issuing warp for both was
// measured to be the bottleneck: a few hundred dependent scalar instructions per iteration at one every
// 4-8 clocks). The producer and issuing warps stay
// converged and issue through one elected lane with predicated instructions and warp-uniform operands:
// issued from inside a divergent branch, a TMA copy or an MMA cost 90-200 clocks each here and the
// issuing thread was the bottleneck; this way they cost 25-35. S and P are double-buffered:
//   S warp:     S(j) as soon as stage j has landed and softmax(j-2) has loaded S(j-2) into registers
//               (bar_sfree; e4m3: P(j-3) . V has completed, bar_buf) -> commit(bar_s[j&1])
//   PV warp:    wait bar_p[i&1] -> PV(i), l(i) -> commit(stage empty), commit(bar_pv[i&1])
//   softmax:    wait bar_s[i&1] -> tcgen05.ld S -> arrive(bar_sfree) -> mask (boundary tiles), row max
//               of the raw scores -> running max of iteration i-1 from the other set (bar_m, shared
//               memory) -> publish the new one -> (rarely, after waiting for PV(i-1)) rescale O and l in
//               TMEM when the max grew by more than 2^8 -> wait PV(i-2) (P buffer free) -> P =
//               exp2(S * scale - ref) as bf16 pairs (packed f32x2 FMA, one exp2 per element) ->
//               tcgen05.st P -> arrive(bar_p[i&1])
// e4m3 KV: the tensor core has no bf16 x e4m3 mode, so the products run as e4m3 x e4m3 (kind::f8f6f4,
// K = 32) on the tiles as they lie in the cache, and Q and P are each written as two 8-bit parts, one
// more MMA per part into the same accumulator:
//   Q = hi + lo, both e4m3, after a per-row power of two that brings the row's largest magnitude into
//       [128, 256) (it goes into the row's score constant): 2 x 4 MMAs M128 x N64 x K32 per iteration
//   P = hi (e4m3) + mid (e4m3) + lo (e5m2), each the rounded remainder of the one before: together they
//       are the weight rounded to f16, exactly, for weights down to 2^-6 (the reference maximum is kept
//       2^4 below the row's largest score, so that is 2^-10 of the largest weight); 3 x 2 MMAs
//       M128 x N128 x K32, a step spanning two pages whose V tiles are contiguous. Two parts (2^-7
//       relative) were not enough: with page scales spread over many powers of two an output element
//       could miss 2e-2 + 2e-2 |ref| by cancellation.
//   S(it) and P(it) share one of three 64-column buffers (it % 3): P is written over the scores it came
//       from, and S(it + 3) follows once P(it) . V has completed (bar_buf).
// The page scales stay out of the tiles: the K scale is the score factor of the page's 16 columns; the V
// scale enters as log2(v_scale) added to the score, so that P carries it into P . V_raw, and each page's
// sum of P divided by v_scale is its share of the row sum, which the softmax warps keep in registers.
// Each softmax set has an O of its own (and its own running maximum and row sum), merged at the end
// like split-KV partials, so the sets exchange nothing per iteration. A twelfth, idle warp completes
// the third warpgroup so that setmaxnreg can move registers from the control warps to the softmax warps.
// All mbarrier waits are bounded; TMEM is always released before the CTA exits.
#include <type_traits>

#include "common.cuh"
#include "tma_ptx.cuh"
#include "tcgen05_ptx.cuh"

namespace pda {

namespace {

constexpr int kTcRows = kUmmaRows;      // query rows per CTA (UMMA M)
constexpr int kTcPagesPerIter = 4;      // 64 tokens per iteration
constexpr int kTcOnesBytes = 2048;                         // bf16 ones: B operand [16 tokens][16 columns] of the row-sum MMA
constexpr int kTcMBytes = 2 * kTcRows * 4;                 // running row maxima handed between the two softmax sets
constexpr int kTcRowBytes = 3 * kTcRows * 4;               // e4m3: per-row score constant, the two sets' row sums
// Sizes that depend on head_dim D (128 or 64) and on the cache's element size (e4m3: D = 128). A row of
// the cache is D * element size / 128 lines of 128 bytes. An operand block = what the tensor core reads
// for one iteration and what one ring stage holds: K of 4 pages as [lines][64 tokens][128 B], then 4 V
// page tiles.
template <int D, bool kFp8>
struct TcCfg {
  static_assert(!kFp8 || D == 128, "e4m3 is built for head_dim 128");
  static constexpr int kElemBytes = kFp8 ? 1 : 2;
  static constexpr int kLines = D * kElemBytes / 128;
  static constexpr int kTileBytes = kPageSize * D * kElemBytes;  // one K or V page tile: 4096 / 2048 (bf16), 2048 (e4m3)
  static constexpr int kKBytes = kTcPagesPerIter * kTileBytes;   // K of 4 pages as [lines][64 tokens][128 B]
  static constexpr int kOperandBytes = 2 * kKBytes;              // K block, then 4 V page tiles: 32 / 16 KB
  static constexpr int kStageBytes = kOperandBytes;
  static constexpr int kStages = 192 * 1024 / kStageBytes;       // 192 KB in flight per SM
  static constexpr int kScaleBytes = kFp8 ? kStages * 16 * 4 : 0;  // per stage and page: score factor, log2 and 1 / V scale
  static constexpr int kSmemBytes = kStages * kStageBytes + kTcOnesBytes + kTcMBytes + kTcRowBytes + kScaleBytes +
                                    512 + 1024;
  // warps: softmax 0-7, producer, S issue (+ TMEM allocation), PV issue
  static constexpr int kProducerWarp = 8, kMmaWarp = 9, kPvWarp = 10;
  // e4m3: a twelfth, idle warp completes the third warpgroup, whose registers go to the softmax warps
  static constexpr int kThreads = kFp8 ? 384 : 352;
};
constexpr int kTcSoftmaxWarps = 8;      // two sets of 4: set x takes the iterations it with it % 2 == x
// e4m3: three warpgroups start with 168 registers a thread; the control group keeps 72 and each softmax
// group takes 208 (setmaxnreg): 2 x 128 x 208 + 128 x 72 <= 65536. With 168 the softmax loop spilled.
constexpr uint32_t kTcRegsSoftmax = 208, kTcRegsControl = 72;
// Tensor memory columns (32-bit each, 128 lanes = query rows), bf16: S buffers 0..63 and 64..127 (f32),
// O 128..255 (f32), Q 256..319 (bf16 pairs along d), P buffers 320..351 and 352..383 (bf16 pairs along
// tokens), l 384..399. Allocations are powers of two.
// e4m3: three S / P buffers 0..63, 64..127, 128..191 (iteration it uses it % 3: S as 64 f32 columns, then P
// over it, four tokens to a column: 16 columns each of high, middle and low parts); each softmax set
// accumulates into an O of its own (192..319 and 320..447); Q 448..511 (four elements to a column: 32
// columns of high parts, then 32 of low parts).
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemL = 384;  // l (bf16): row sums of P, 16 columns (all equal)
template <bool kFp8> constexpr uint32_t kTmemO = kFp8 ? 192 : 128;
template <bool kFp8> constexpr uint32_t kTmemQ = kFp8 ? 448 : 256;
constexpr uint32_t kTmemPBf16 = 320;
constexpr int kFp8Bufs = 3;
constexpr float kRescaleThreshold = 8.f;  // log2 units: O is rescaled only when the max grows this much
// e4m3: the reference is set this far below the largest score seen (log2 units), so that the weights start
// at 2^4 and may grow to 2^8 before a rescale: the three 8-bit parts of a weight are exact from 2^-6 up.
constexpr float kFp8RefBelowMax = 4.f;

template <int D, bool kFp8>
__global__ void __launch_bounds__((TcCfg<D, kFp8>::kThreads), 1)
attention_mq_tc_kernel(const __grid_constant__ CUtensorMap k_map,
                       const __grid_constant__ CUtensorMap v_map, MqParams mp) {
  const AttnParams& p = mp.a;
  using C = TcCfg<D, kFp8>;
  constexpr int kTcStages = C::kStages, kTcStageBytes = C::kStageBytes, kTcKBytes = C::kKBytes,
                kTcTileBytes = C::kTileBytes, kTcThreads = C::kThreads;
  constexpr int kTcProducerWarp = C::kProducerWarp, kTcMmaWarp = C::kMmaWarp, kTcPvWarp = C::kPvWarp;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ones_smem = smem + kTcStages * kTcStageBytes;
  float* m_sh = reinterpret_cast<float*>(ones_smem + kTcOnesBytes);        // [2][128]
  float* rowc_sh = m_sh + 2 * kTcRows;                                     // e4m3: [128] score constant of the row
  float* l_sh = rowc_sh + kTcRows;                                         // e4m3: [2][128] the sets' row sums
  float* scale_sh = l_sh + 2 * kTcRows;                                    // e4m3: [stage][4 c, 4 a, 4 1/v, 4 unused]
  // full[], empty[], s[2], p[2], pv[2], sfree[2], m[2][4], buf[3] (+1 unused), s3[3] (+1 unused)
  uint64_t* bars = reinterpret_cast<uint64_t*>(ones_smem + kTcOnesBytes + kTcMBytes + kTcRowBytes + C::kScaleBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kTcStages + 24);
  int* cta_err = reinterpret_cast<int*>(tmem_slot + 1);
  int* rank_slot = cta_err + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.group, T = mp.n_q;
  const int rows_total = T * G;
  const int n_rb = (rows_total + kTcRows - 1) / kTcRows;
  const int c = blockIdx.x, g = blockIdx.y / n_rb, rb = blockIdx.y % n_rb;
  const bool split = p.chunk_tokens > 0;
  // unsplit units differ in length: the CTA with blockIdx.z = r serves the r-th longest sequence
  const bool ranked = !split && mp.kv_len_fixed == 0 && p.batch > 1 && p.batch <= 128;
  int b = blockIdx.z;
  // Everything below up to the roles is the serial start of the CTA (about 5 us before the first P): the
  // set-up that does not depend on the sequence comes first and shares its barrier with the ranking.
  // (the loads of the status word and of the lengths are issued together: each is a trip to L2 or DRAM)
  const int32_t status_now = p.status != nullptr ? *reinterpret_cast<volatile int32_t*>(p.status) : 0;
  int len_mine = 0;  // ranked: the length of sequence tid
  if (ranked && tid < p.batch) len_mine = max(p.seq_lens[tid], 0);
  if (split) {  // an empty chunk leaves before anything is allocated
    const int Lb = mp.kv_len_fixed > 0 ? mp.kv_len_fixed : max(p.seq_lens[b], 0);
    if (p.first_token + c * p.chunk_tokens >= Lb) return;
  }
  // once any CTA of this launch has reported a timed-out wait, the rest do not start
  if (status_now == PDA_DEV_TIMEOUT) return;

  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kTcStages;
  const uint32_t bar_s = empty0 + 8 * kTcStages, bar_p = bar_s + 16, bar_pv = bar_p + 16;  // two of each
  const uint32_t bar_sfree = bar_pv + 16, bar_m = bar_sfree + 16;
  const uint32_t bar_buf = bar_m + 64;  // e4m3: S / P buffer k is free again (its P . V has completed)
  // e4m3: S is ready in buffer k. One barrier per BUFFER, not per softmax set: the next S into a buffer needs
  // the P . V of the one before, hence the softmax of the one before, so a barrier is never completed twice
  // before its waiter has looked (with one per set, S(it + 2) -- which waits for no softmax warp here -- could
  // complete the set's barrier a second time while the set had not yet waited for S(it), and a parity wait
  // cannot tell phases two apart: a set was then left waiting for good)
  const uint32_t bar_s3 = bar_buf + 32;
  if constexpr (!kFp8) {
    for (int i = tid; i < kTcOnesBytes / 4; i += kTcThreads)
      reinterpret_cast<uint32_t*>(ones_smem)[i] = 0x3F803F80u;  // 1.0 as bf16 pairs
    fence_proxy_async();  // read by the tensor core through the async proxy
  }
  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);  // released by the PV MMAs' commit
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(bar_s + 8 * k, 1);
      mbar_init(bar_p + 8 * k, 4);   // one arrival per warp of the softmax set that owns the iteration
      mbar_init(bar_pv + 8 * k, 1);
      mbar_init(bar_sfree + 8 * k, 4);
#pragma unroll
      for (int w = 0; w < 4; ++w) mbar_init(bar_m + 8 * (4 * k + w), 1);  // per warp: rows w*32.. of set k
    }
    for (int k = 0; k < kFp8Bufs; ++k) {
      mbar_init(bar_buf + 8 * k, 1);
      mbar_init(bar_s3 + 8 * k, 1);
    }
    *cta_err = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == kTcMmaWarp) {  // tensor memory; this warp also releases it
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (ranked) {
    int* lens = reinterpret_cast<int*>(smem);  // (aliases the ring, which nothing writes before the barrier below)
    if (tid < p.batch) lens[tid] = len_mine;  // (batch <= 128 < threads)
    __syncthreads();
    // rank of sequence j = how many come before it (longer, or as long with a lower index); `parts` lanes
    // share a sequence's comparisons
    int parts = 1;
    while (parts < 32 && parts * 2 * p.batch <= kTcThreads) parts *= 2;
    const int j = tid / parts, part = tid % parts;
    int rank = 0;
    if (j < p.batch) {
      const int Lj = lens[j];
      for (int i = part; i < p.batch; i += parts) rank += (lens[i] > Lj) || (lens[i] == Lj && i < j);
    }
    for (int o = 1; o < parts; o <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
    if (j < p.batch && part == 0 && rank == static_cast<int>(blockIdx.z)) {
      rank_slot[0] = j;
      rank_slot[1] = lens[j];
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (ranked) b = rank_slot[0];

  const int L = mp.kv_len_fixed > 0 ? mp.kv_len_fixed : ranked ? rank_slot[1] : max(p.seq_lens[b], 0);
  int t0 = p.first_token, t1 = L;
  if (split) {
    t0 = p.first_token + c * p.chunk_tokens;
    t1 = min(t0 + p.chunk_tokens, L);
  }
  int err = 0;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ||
      (split && static_cast<int64_t>(L - p.first_token) >
                    static_cast<int64_t>(p.max_chunks - p.chunk_slot0) * p.chunk_tokens))
    err = PDA_DEV_BAD_SEQ_LEN;
  const int page0 = t0 / kPageSize;
  const int n_pages = err ? 0 : (t1 + kPageSize - 1) / kPageSize - page0;
  const int n_iters = (n_pages + kTcPagesPerIter - 1) / kTcPagesPerIter;

  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + kTmemO<kFp8>;  // S buffer k at tmem_s + 64 k
  const uint32_t tmem_q = tmem_base + kTmemQ<kFp8>;
  const uint32_t tmem_p = tmem_base + kTmemPBf16;  // bf16: P buffer k at tmem_p + 32 k (e4m3: P lies over its S)

  const int32_t* table = p.block_table + static_cast<int64_t>(b) * p.block_table_stride;
  // e4m3, at most 64 query rows (e.g. 16 draft tokens x a group of 4): every row is held twice, in TMEM
  // lanes r and r + 64, and the two copies share the softmax work of an iteration -- lane r takes its
  // first 32 tokens, lane r + 64 the other 32, each as an online softmax of its own (own maximum, own row
  // sum, own accumulator lane; the other half of its P is zero), merged at the end like split-KV partials.
  // The softmax warps' chain per iteration, which bounds this kernel, is then half as long.
  const bool half_rows = kFp8 && rows_total <= kTcRows / 2;

  // The roles, as closures.
  // ---- Q: row r -> (query token r / G, head r % G) goes to TMEM lane r as the A operand of S = Q . K^T
  auto load_q = [&]() {
    // the two softmax warps that own the same 32 rows (w and w + 4) take half a row each
    if (warp < kTcSoftmaxWarps && (warp >> 2) < D / 64) {
      const int t = tid & (kTcRows - 1), half = warp >> 2;
      const int r = half_rows ? (t & (kTcRows / 2 - 1)) : rb * kTcRows + t;
      const bool valid = r < rows_total;
      const int64_t qrow = (static_cast<int64_t>(b) * T + r / G) * p.num_q_heads + g * G + (r % G);
      const uint4* src = reinterpret_cast<const uint4*>(p.q + qrow * D);
      const uint32_t my_q = tmem_q + (static_cast<uint32_t>((warp & 3) * 32) << 16);
      if constexpr (!kFp8) {
        uint32_t qv[32];  // 64 bf16 = 32 columns
  #pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          const uint4 v = valid ? src[half * 8 + ch] : make_uint4(0u, 0u, 0u, 0u);
          qv[4 * ch] = v.x; qv[4 * ch + 1] = v.y; qv[4 * ch + 2] = v.z; qv[4 * ch + 3] = v.w;
        }
        tmem_st32(my_q + 32 * half, qv);
      } else {
        // e4m3 x e4m3 on the tensor core: the row is scaled by a power of two so that its largest
        // magnitude lies in [128, 256) and written as hi + lo, both e4m3 (|q - hi - lo| <= 2^-8 |q| or
        // 2^-17 of the row's largest magnitude); the power of two goes into the row's score constant.
        // (Both warps read the whole row for the magnitude; each converts its half.)
        uint32_t qw[D / 4];
        uint32_t amax = 0u;  // bf16 magnitudes order like their bit patterns
  #pragma unroll
        for (int ch = 0; ch < D / 8; ++ch) {
          const uint4 v = valid ? src[ch] : make_uint4(0u, 0u, 0u, 0u);
          const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
  #pragma unroll
          for (int e = 0; e < 4; ++e) {
            amax = max(amax, max((w4[e] << 16) & 0x7fff0000u, w4[e] & 0x7fff0000u));
            if ((ch >> 3) == half) qw[4 * (ch & 7) + e] = w4[e];
          }
        }
        const int ex = static_cast<int>(amax >> 23);                      // biased exponent of the largest magnitude
        const int up = (ex == 0 || ex == 255) ? 0 : min(max(134 - ex, -100), 100);  // it times 2^up is in [128, 256)
        const float mul = __uint_as_float(static_cast<uint32_t>(127 + up) << 23);
        if (half == 0) rowc_sh[t] = p.scale * 1.4426950408889634f * __uint_as_float(static_cast<uint32_t>(127 - up) << 23);
        uint32_t qh[16], ql[16];
  #pragma unroll
        for (int c4 = 0; c4 < D / 8; ++c4) {  // four elements -> one 32-bit column of each part
          uint32_t h2[2], l2[2];
  #pragma unroll
          for (int e = 0; e < 2; ++e) {
            const uint32_t w = qw[2 * c4 + e];
            const float x0 = __uint_as_float(w << 16) * mul, x1 = __uint_as_float(w & 0xffff0000u) * mul;
            h2[e] = f32x2_to_e4m3x2(x0, x1);
            uint32_t back16 = e4m3x2_to_f16x2(h2[e]);  // what the tensor core will read for the high parts
            const float2 back = __half22float2(*reinterpret_cast<__half2*>(&back16));
            l2[e] = f32x2_to_e4m3x2(x0 - back.x, x1 - back.y);
          }
          qh[c4] = h2[0] | (h2[1] << 16);
          ql[c4] = l2[0] | (l2[1] << 16);
        }
        tmem_st16(my_q + 16 * half, qh);
        tmem_st16(my_q + 32 + 16 * half, ql);
      }
      tmem_wait_st();
    }
  };
  auto wait_q = [&]() {
    // Q is in tensor memory before the first MMA is issued (the producer does not take part)
    tc_fence_before();
    asm volatile("bar.sync 1, %0;" ::"n"(kTcThreads - 32) : "memory");
    tc_fence_after();
  };
  auto producer_role = [&]() {
    // ================= TMA producer (does not wait for Q) =================
    const uint32_t leader = elect_one();
    const int u_iters = __shfl_sync(0xffffffffu, n_iters, 0);
    const int u_pages = __shfl_sync(0xffffffffu, n_pages, 0);
    bool bad = false;
    int pg = 0;
    // e4m3, per page: the score factor (K scale), log2 of the V scale and its reciprocal. The scales are
    // positive by construction; the clamps keep an all-zero or negative entry from producing inf or NaN.
    // (lanes past the last page keep finite values: a masked score times 0 would be NaN)
    float sc_c = 1.f, sc_a = 0.f, sc_i = 1.f;
    for (int it = 0; it < u_iters; ++it) {
      const int s = it % kTcStages;
      if ((it & 7) == 0) {  // page ids of the next 8 iterations (32 pages), one per lane
        pg = 0;
        if (it * kTcPagesPerIter + lane < u_pages) {
          const int v = table[page0 + it * kTcPagesPerIter + lane];
          pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
          if (kFp8) {
            const float ks = fabsf(p.k_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g]);
            const float vs = fabsf(p.v_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g]);
            const float vc = fminf(fmaxf(vs, 8.6736174e-19f), 1.1529215e18f);  // 2^-60 .. 2^60
            sc_c = fminf(fmaxf(ks, 1e-30f), 1e30f);
            sc_a = __log2f(vc);
            sc_i = 1.f / vc;
          }
        }
      }
      bool ok = true;
      if (it >= kTcStages) ok = mbar_wait_bounded(empty0 + 8 * s, ((it / kTcStages) - 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); break; }
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      const uint32_t stage = ring + s * kTcStageBytes, bar = full0 + 8 * s;
      if (kFp8) {  // this stage's page constants, written by the lanes that hold its pages (seen through the full barrier)
        if ((lane >> 2) == (it & 7)) {
          scale_sh[s * 16 + (lane & 3)] = sc_c;
          scale_sh[s * 16 + 4 + (lane & 3)] = sc_a;
          scale_sh[s * 16 + 8 + (lane & 3)] = sc_i;
        }
        __syncwarp();
      }
      mbar_expect_tx_if(leader, bar, n_here * 2 * kTcTileBytes);
      // K: one copy per 128-byte line so that page j's 16 rows follow page j-1's in each line block
      // (an e4m3 row is one line)
      auto load_page = [&](int j) {
        const int page_raw = __shfl_sync(0xffffffffu, pg, (it & 7) * kTcPagesPerIter + j);
        bad |= page_raw < 0;
        const int page = max(page_raw, 0);
#pragma unroll
        for (int ln = 0; ln < C::kLines; ++ln)
          tma_load_5d_if(leader, stage + ln * (kTcKBytes / C::kLines) + j * (kPageSize * 128), &k_map, bar, ln, g, page);
        tma_load_5d_if(leader, stage + kTcKBytes + j * kTcTileBytes, &v_map, bar, 0, g, page);
      };
      if (n_here == kTcPagesPerIter) {
#pragma unroll
        for (int j = 0; j < kTcPagesPerIter; ++j) load_page(j);
      } else {
        for (int j = 0; j < n_here; ++j) load_page(j);
      }
    }
    if (bad && lane == 0) atomicMax(cta_err, PDA_DEV_BAD_PAGE);
  };
  auto s_issue_role = [&]() {
    // ================= S issue: S(it) = Q . K^T as soon as its operands allow =================
    // (Two issuing warps, one for S and one for PV: a single warp runs the few hundred dependent scalar
    // instructions of both per iteration at one every 4-8 clocks, which is as long as the iteration
    // itself. Each keeps to its own chain of barriers; the tensor core's order between the two does not
    // matter.)
    constexpr uint32_t idesc_s = kFp8 ? tc_idesc(kTcPagesPerIter * kPageSize, false, kFmtE4m3, kFmtE4m3)
                                      : tc_idesc(kTcPagesPerIter * kPageSize, false, kFmtBf16, kFmtBf16);
    const uint32_t leader = elect_one();
    // warp-uniform copies (a shuffle from lane 0 tells the compiler so)
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    const int u_iters = __shfl_sync(0xffffffffu, n_iters, 0);
    const int u_pages = __shfl_sync(0xffffffffu, n_pages, 0);
    const int u_tail0 = __shfl_sync(0xffffffffu, L - page0 * kPageSize, 0);  // tokens from the first page to the end
    bool ok = true;
    uint32_t stage_i = 0, stage_par = 0;  // the iteration's ring stage and the phase parity of its full barrier
    uint32_t buf_i = 0, buf_round = 0;    // e4m3: it % 3 and it / 3
    for (int it = 0; it < u_iters; ++it) {
      if constexpr (kFp8) {
        // (the stage first: it has landed long ago as a rule, while the buffer is what S waits for)
        ok = mbar_wait_bounded(full0 + 8 * stage_i, stage_par);  // the block has landed
        // S(it) overwrites the buffer of S(it-3) and P(it-3): P(it-3) . V has completed
        if (ok && it >= kFp8Bufs) ok = mbar_wait_bounded(bar_buf + 8 * buf_i, (buf_round - 1) & 1);
      } else {
        // S(it) overwrites the buffer of S(it-2): the softmax warps have loaded that into registers
        if (it >= 2) ok = mbar_wait_bounded(bar_sfree + 8 * (it & 1), ((it - 2) >> 1) & 1);
        if (ok) ok = mbar_wait_bounded(full0 + 8 * stage_i, stage_par);  // the block has landed
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t stage = ring + stage_i * C::kOperandBytes;
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      const int tail = u_tail0 - (it * kTcPagesPerIter + n_here - 1) * kPageSize;  // valid rows of the last page here
      // P is 0 past the sequence end, but V must be finite there: clear those rows of the last page, and
      // (e4m3, where an MMA step spans two pages) the missing second page of the last step
      const bool odd = kFp8 && (n_here & 1);
      if (tail < kPageSize || odd) {
        const uint32_t vt = stage + kTcKBytes + (n_here - 1) * kTcTileBytes;
        if constexpr (kFp8) {  // a row is one 128-byte line: the rows to clear are contiguous
          const int first = max(min(tail, kPageSize), 0) * 128, end = (odd ? 2 : 1) * kTcTileBytes;
          for (int i = first + lane * 16; i < end; i += 32 * 16)
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + i), "r"(0));
        } else {
          constexpr int kChunksPerRow = D / 8;  // 16-byte chunks of a row
          for (int i = lane; i < (kPageSize - tail) * kChunksPerRow; i += 32) {
            const int r = tail + i / kChunksPerRow, ch = i % kChunksPerRow;
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_off(r, ch)), "r"(0));
          }
        }
        fence_proxy_async();
        __syncwarp();
      }
      tc_fence_after();
      const uint32_t d = u_tmem + 64 * (kFp8 ? buf_i : static_cast<uint32_t>(it & 1));
      // S[:, 0..64) = Q . K^T over the 64 stacked token rows
      // (rows of pages that were not loaded hold stale data: those columns are masked later)
      const uint64_t kd0 = tc_desc(stage, 16, 1024);
      if constexpr (kFp8) {
        // contraction over d in 4 steps of 32, once with the high and once with the low parts of Q;
        // descriptor start addresses are in 16-byte units: +2 per k-step of 32 bytes
#pragma unroll
        for (int part = 0; part < 2; ++part)
#pragma unroll
          for (int ks = 0; ks < D / 32; ++ks)
            tc_mma_ts_if<true>(leader, d, u_tmem + kTmemQ<true> + 32 * part + 8 * ks, kd0 + static_cast<uint64_t>(ks * 2),
                               idesc_s, (part | ks) ? 1u : 0u);
      } else {
        // contraction over d in steps of 16
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          // +2 per k-step, next line block further on
          const uint64_t bd = kd0 + static_cast<uint64_t>((ks >> 2) * (kTcKBytes / C::kLines / 16) + (ks & 3) * 2);
          tc_mma_ts_if<false>(leader, d, u_tmem + kTmemQ<false> + 8 * ks, bd, idesc_s, ks > 0 ? 1u : 0u);
        }
      }
      tc_commit_if(leader, kFp8 ? bar_s3 + 8 * buf_i : bar_s + 8 * (it & 1));
      if (++stage_i == kTcStages) { stage_i = 0; stage_par ^= 1; }
      if (++buf_i == kFp8Bufs) { buf_i = 0; ++buf_round; }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };
  auto pv_issue_role = [&]() {
    // ================= PV issue: O += P . V and l += P . 1 =================
    constexpr uint32_t idesc_pv = kFp8 ? tc_idesc(D, true, kFmtE4m3, kFmtE4m3) : tc_idesc(D, true, kFmtBf16, kFmtBf16);
    constexpr uint32_t idesc_pv_lo = tc_idesc(D, true, kFmtE5m2, kFmtE4m3);  // e4m3 caches: the low parts of P are e5m2
    constexpr uint32_t idesc_l = tc_idesc(16, false, kFmtBf16, kFmtBf16);
    const uint64_t ones_desc = tc_desc(smem_u32(ones_smem), 16, 1024);
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    const int u_iters = __shfl_sync(0xffffffffu, n_iters, 0);
    const int u_pages = __shfl_sync(0xffffffffu, n_pages, 0);
    bool ok = true;
    uint32_t stage_i = 0;  // the iteration's ring stage
    uint32_t buf_i = 0;    // e4m3: it % 3
    for (int it = 0; it < u_iters; ++it) {
      ok = mbar_wait_bounded(bar_p + 8 * (it & 1), (it >> 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t stage = ring + stage_i * C::kOperandBytes;
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      const uint32_t pa0 = kFp8 ? u_tmem + 64 * buf_i : u_tmem + kTmemPBf16 + 32 * (it & 1);
      // V read MN-major. LBO: next 64 columns of d (bf16; an e4m3 line holds all 128), SBO: next 8 tokens
      const uint64_t vd0 = tc_desc(stage + kTcKBytes, kPageSize * 128, 1024);
      if constexpr (kFp8) {
        // O[it % 2] += P[:, 32j .. 32j+32) . V : one K = 32 step per two pages (their tiles are contiguous),
        // once with each of the three parts of P (high, middle: e4m3; low: e5m2); the row sums are kept by
        // the softmax warps
        auto pv_pair = [&](int j) {
#pragma unroll
          for (int part = 0; part < 3; ++part)
            tc_mma_ts_if<true>(leader, u_tmem + kTmemO<true> + D * (it & 1), pa0 + 16 * part + 8 * j,
                               vd0 + static_cast<uint64_t>(j * (2 * kTcTileBytes / 16)), part == 2 ? idesc_pv_lo : idesc_pv,
                               (it > 1 || j > 0 || part > 0) ? 1u : 0u);
        };
        pv_pair(0);
        if (n_here > 2) pv_pair(1);
      } else {
        // O += P[:, 16j .. 16j+16) . V_j : one K = 16 step per page
        // and l += P[:, 16j .. 16j+16) . 1 : the row sums of exactly the P that multiplies V
        auto pv_page = [&](int j) {
          const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
          tc_mma_ts_if<false>(leader, u_tmem + kTmemO<false>, pa0 + 8 * j, vd0 + static_cast<uint64_t>(j * (kTcTileBytes / 16)), idesc_pv, acc);
          tc_mma_ts_if<false>(leader, u_tmem + kTmemL, pa0 + 8 * j, ones_desc, idesc_l, acc);
        };
        if (n_here == kTcPagesPerIter) {
#pragma unroll
          for (int j = 0; j < kTcPagesPerIter; ++j) pv_page(j);
        } else {
          for (int j = 0; j < n_here; ++j) pv_page(j);
        }
      }
      tc_commit_if(leader, empty0 + 8 * stage_i);     // the stage may be refilled once these MMAs have read it
      tc_commit_if(leader, bar_pv + 8 * (it & 1));    // O (and l) updated, P buffer free again
      if constexpr (kFp8) tc_commit_if(leader, bar_buf + 8 * buf_i);  // ... which the S issue warp waits for
      if (++stage_i == kTcStages) stage_i = 0;
      if (++buf_i == kFp8Bufs) buf_i = 0;
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };
  auto softmax_role = [&]() {
    // ================= softmax on bf16 caches: TMEM lane t <-> query row t; set x takes iterations x, x+2, ...
    // Two warps per scheduler, one of each set: while one waits (for S, for the other set's row maximum,
    // for its tcgen05.ld/st) the other keeps the exp2 unit busy, which is what bounds this part.
    const int set = warp >> 2, t = tid & (kTcRows - 1);
    const int r = rb * kTcRows + t;
    const int i_tok = r / G;
    const int lim = mp.causal ? min(L, L - T + i_tok + 1) : L;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;  // this warp's TMEM lanes
    const float scale_log2 = p.scale * 1.4426950408889634f;
    const uint32_t my_s = bar_s + 8 * set, my_p = bar_p + 8 * set, my_pv = bar_pv + 8 * set;
    const uint32_t my_sfree = bar_sfree + 8 * set;
    // the running maximum passes between the two warps that own the same 32 rows (same scheduler)
    const uint32_t my_m = bar_m + 8 * (4 * set + (warp & 3)), other_m = bar_m + 8 * (4 * (set ^ 1) + (warp & 3));
    float m_ref = -INFINITY;   // reference max the accumulated O and l are scaled by
    bool alive = true;
    auto fail = [&]() { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); alive = false; };
    for (int it = set; it < n_iters; it += 2) {
      const int k = it >> 1;  // this set's k-th iteration: the phase index of its barriers
      bool ok = mbar_spin_bounded(my_s, k & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { fail(); break; }
      tc_fence_after();
      uint32_t sv[2][32];
      tmem_ld32(tmem_s + 64 * set + lane_base, sv[0]);
      tmem_ld32(tmem_s + 64 * set + lane_base + 32, sv[1]);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_tc(my_sfree);  // S(it) is in registers: S(it+2) may overwrite its buffer
      const int tok0 = (page0 + it * kTcPagesPerIter) * kPageSize;
      const int n_vis = min(lim, t1) - tok0;  // visible columns of this row in this iteration (may be <= 0)
      if (__any_sync(0xffffffffu, n_vis < kTcPagesPerIter * kPageSize)) {  // boundary tiles only
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int j = 0; j < 32; ++j)
            sv[h][j] = (h * 32 + j < n_vis) ? sv[h][j] : 0xff800000u;  // -inf
      }
      // row maximum of the raw scores (the scale is positive), four independent chains
      float mxs[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < 32; j += 2)
          mxs[(j >> 1) & 3] = max3(mxs[(j >> 1) & 3], __uint_as_float(sv[h][j]), __uint_as_float(sv[h][j + 1]));
      const float mx = fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])) * scale_log2;
      // the reference after iteration it-1 comes from the other set (one O for both)
      if (it > 0) {
        ok = mbar_spin_bounded(other_m, ((it - 1) >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        m_ref = m_sh[((it - 1) & 1) * kTcRows + t];
      }
      // lazy rescaling: keep the old reference unless the max grew past the threshold
      float m_new = m_ref;
      if (mx > m_ref + kRescaleThreshold || m_ref == -INFINITY) m_new = fmaxf(m_ref, mx);
      const bool need = m_new != m_ref && m_ref != -INFINITY;
      m_sh[(it & 1) * kTcRows + t] = m_new;
      __syncwarp();
      if (lane == 0) mbar_arrive_tc(my_m);  // (release: the other set reads m_sh after its wait)
      if (it > 0 && __any_sync(0xffffffffu, need)) {
        // O and l may only be touched once the last PV into them, PV(it-1), has completed. PV(it) is not
        // issued before this warp arrives on bar_p below, and the other set rescales only after PV(it)
        // (a parity wait tells neighbouring phases apart only: first this set's own PV(it-2), after which
        // the other set's barrier cannot be more than one phase behind)
        ok = it >= 2 ? mbar_spin_bounded(my_pv, (k - 1) & 1) : true;
        if (ok) ok = mbar_spin_bounded(bar_pv + 8 * (set ^ 1), ((it - 1) >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        const float alpha = need ? ex2(m_ref - m_new) : 1.f;
        const uint32_t my_o = tmem_o + lane_base;
#pragma unroll
        for (int cb = 0; cb < D / 32 + 1; ++cb) {  // O, then the block of columns that holds l
          uint32_t ov[32];
          tmem_ld32(my_o + (cb < D / 32 ? 32 * cb : kTmemL - kTmemO<false>), ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
          tmem_st32(my_o + (cb < D / 32 ? 32 * cb : kTmemL - kTmemO<false>), ov);
        }
        tmem_wait_st();
      }
      m_ref = m_new;
      const float ref = m_ref == -INFINITY ? 0.f : m_ref;
      uint32_t pw[32];
      {
        // P = exp2(S * scale_log2 - ref) as bf16 pairs into TMEM lane t: the A operand of O += P . V
        // (one packed FMA per two elements; masked columns stay -inf -> 0)
        const uint64_t c2 = f32x2(__float_as_uint(scale_log2), __float_as_uint(scale_log2));
        const uint64_t nr2 = f32x2(__float_as_uint(-ref), __float_as_uint(-ref));
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const uint64_t x2 = fma_f32x2(f32x2(sv[j >> 4][(2 * j) & 31], sv[j >> 4][(2 * j + 1) & 31]), c2, nr2);
          float x0, x1;
          f32x2_split(x2, x0, x1);
          pw[j] = pack2<false>(ex2(x0), ex2(x1));
        }
      }
      if (it >= 2) {  // PV(it-2) has finished reading the P buffer this iteration writes
        ok = mbar_spin_bounded(my_pv, (k - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
      }
      tmem_st32(tmem_p + 32 * set + lane_base, pw);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_tc(my_p);
    }

    // ---- finalise: the last iteration's reference (from the set that owned it) and the last PV
    bool ok = alive;
    if (alive && n_iters > 0) {
      const int last = n_iters - 1;
      if ((last & 1) != set) {
        ok = mbar_spin_bounded(bar_m + 8 * (4 * (last & 1) + (warp & 3)), (last >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) m_ref = m_sh[(last & 1) * kTcRows + t];
      }
      if (ok) {
        // (the set that does not own the last iteration waits for its own last PV first: see above)
        if ((last & 1) != set && last >= 1) ok = mbar_wait_bounded(my_pv, ((last - 1) >> 1) & 1);
        if (ok) ok = mbar_wait_bounded(bar_pv + 8 * (last & 1), (last >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
      }
      if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
      tc_fence_after();
    }
    // every softmax warp reaches this point together with its error view settled
    asm volatile("bar.sync 2, %0;" ::"n"(kTcSoftmaxWarps * 32) : "memory");
    const int dev_err = max(err, *cta_err);
    if (dev_err && tid == 0) report(p.status, dev_err);
    const bool valid_row = r < rows_total;
    const bool have = alive && ok && n_iters > 0;  // warp-uniform
    float l = 0.f;
    if (have) {
      uint32_t lv[32];
      tmem_ld32(tmem_base + kTmemL + lane_base, lv);
      tmem_wait_ld();
      l = __uint_as_float(lv[0]);
    }
    const bool live = !dev_err && have && l > 0.f;
    const float inv = live ? 1.f / l : 0.f;
    const int64_t qrow = (static_cast<int64_t>(b) * T + i_tok) * p.num_q_heads + g * G + (r % G);
    constexpr float kLn2 = 0.6931471805599453f;
    // set x stores columns [D/2 x, D/2 (x + 1)) of the row, 32 at a time
#pragma unroll
    for (int cb = (D / 64) * set; cb < (D / 64) * (set + 1); ++cb) {
      uint32_t ov[32];
      if (have) {
        tmem_ld32(tmem_o + lane_base + 32 * cb, ov);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[j] = 0u;
      }
      if (valid_row) {
        if (split) {
          float4* dst = reinterpret_cast<float4*>(p.part_o + (qrow * p.max_chunks + p.chunk_slot0 + c) * D + 32 * cb);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(live ? __uint_as_float(ov[4 * j]) * inv : 0.f, live ? __uint_as_float(ov[4 * j + 1]) * inv : 0.f,
                                 live ? __uint_as_float(ov[4 * j + 2]) * inv : 0.f, live ? __uint_as_float(ov[4 * j + 3]) * inv : 0.f);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(p.out + qrow * D + 32 * cb);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              w[e] = pack2<false>(live ? __uint_as_float(ov[8 * j + 2 * e]) * inv : 0.f,
                                  live ? __uint_as_float(ov[8 * j + 2 * e + 1]) * inv : 0.f);
            dst[j] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
    if (split && valid_row && set == 0)
      p.part_lse[qrow * p.max_chunks + p.chunk_slot0 + c] = live ? (m_ref + __log2f(l)) * kLn2 : -INFINITY;
  };
  auto softmax_role_fp8 = [&](auto pages_tag) {
    // ================= softmax on e4m3 caches. kNp = pages of an iteration a thread works on: 4 (its row
    // sees all 64 tokens) or 2 (half rows: lanes below 64 take tokens 0..31, lanes from 64 tokens 32..63).
    // Each set runs an online softmax of its own over its iterations, with its own O; nothing is
    // exchanged per iteration.
    constexpr int kNp = decltype(pages_tag)::value;
    constexpr bool kHalf = kNp == 2;
    constexpr int kNc = kNp * kPageSize;  // columns (tokens) per thread and iteration
    const int set = warp >> 2, t = tid & (kTcRows - 1);
    const int half = kHalf ? (t >> 6) : 0;  // warp-uniform
    const int r = kHalf ? (t & (kTcRows / 2 - 1)) : rb * kTcRows + t;
    const int i_tok = r / G;
    const int lim = mp.causal ? min(L, L - T + i_tok + 1) : L;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;  // this warp's TMEM lanes
    const uint32_t my_p = bar_p + 8 * set, my_pv = bar_pv + 8 * set;
    float m_ref = -INFINITY;   // reference the accumulated O is scaled by
    // this thread's share of the row sum l (kept here, not in tensor memory) and the reference it is
    // scaled by; the row's score constant (softmax scale, log2 e and the power of two Q was scaled by)
    float l_set = 0.f, m_l = -INFINITY;
    const float rowc = rowc_sh[t];
    uint32_t sc_stage = set % kTcStages;  // ring stage of this set's next iteration
    uint32_t my_buf = set;                 // S / P buffer of this set's next iteration (it % 3)
    bool alive = true;
    auto fail = [&]() { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); alive = false; };
    for (int it = set; it < n_iters; it += 2) {
      const int k = it >> 1;  // this set's k-th iteration: the phase index of its barriers
      bool ok = mbar_spin_bounded(bar_s3 + 8 * my_buf, (static_cast<uint32_t>(it) / kFp8Bufs) & 1);  // S(it), buffer it % 3
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { fail(); break; }
      tc_fence_after();
      uint32_t sv[kNc];
      const uint32_t sp_buf = tmem_s + 64 * my_buf + lane_base;
      if constexpr (kHalf) {
        tmem_ld32(sp_buf + 32 * half, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
      } else {
        tmem_ld32(sp_buf, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(sp_buf + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
      }
      tmem_wait_ld();
      my_buf = my_buf >= 1 ? my_buf - 1 : my_buf + 2;  // (it + 2) % 3
      const int tok0 = (page0 + it * kTcPagesPerIter) * kPageSize + kNc * half;  // first token of this thread's columns
      const int n_vis = min(lim, t1) - tok0;  // visible ones among them (may be <= 0)
      if (__any_sync(0xffffffffu, n_vis < kNc)) {  // boundary tiles only
#pragma unroll
        for (int j = 0; j < kNc; ++j) sv[j] = (j < n_vis) ? sv[j] : 0xff800000u;  // -inf
      }
      // per page j of the thread's columns: x = s cq[j] + aq[j] with cq = K scale x row constant and aq = log2 of
      // the V scale, i.e. the softmax runs on the scores plus log2(V scale): P then carries the V scale
      // into P . V (V is multiplied as raw e4m3), and dividing the page's sum of P by the V scale (iq)
      // gives its share of l.
      // (the constants were written by the producer before the tiles' full barrier completed, which the
      // S issue warp observed before the MMAs whose commit this warp has waited for)
      float cq[kNp], aq[kNp], iq[kNp];
      {
        const float* sc = scale_sh + sc_stage * 16 + kNp * half;
#pragma unroll
        for (int q = 0; q < kNp; ++q) {
          cq[q] = fmaxf(sc[q] * rowc, 1e-37f);  // (kept above zero: a masked score, -inf, times 0 would be NaN)
          aq[q] = sc[4 + q];
          iq[q] = sc[8 + q];
        }
      }
      sc_stage += 2;
      if (sc_stage >= kTcStages) sc_stage -= kTcStages;
      // row maximum of x over the thread's columns: per page the maximum of the raw scores (the factor is
      // positive), two chains each
      float mx = -INFINITY;
#pragma unroll
      for (int q = 0; q < kNp; ++q) {
        float ma = -INFINITY, mb = -INFINITY;
#pragma unroll
        for (int j = 16 * q; j < 16 * q + 16; j += 4) {
          ma = max3(ma, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]));
          mb = max3(mb, __uint_as_float(sv[j + 2]), __uint_as_float(sv[j + 3]));
        }
        mx = fmaxf(mx, fmaf(fmaxf(ma, mb), cq[q], aq[q]));
      }
      // lazy rescaling: keep the old reference unless the max grew past the threshold; a new reference is
      // set kFp8RefBelowMax under the maximum
      float m_new = m_ref;
      if (mx > m_ref + kRescaleThreshold || m_ref == -INFINITY) m_new = mx - kFp8RefBelowMax;
      const bool need = m_new != m_ref && m_ref != -INFINITY;
      if (it > 1 && __any_sync(0xffffffffu, need)) {
        // O may only be touched once this set's last PV into it, PV(it-2), has completed; PV(it) is not
        // issued before this warp arrives on bar_p below
        ok = mbar_spin_bounded(my_pv, (k - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        const float alpha = need ? ex2(m_ref - m_new) : 1.f;
        const uint32_t my_o = tmem_o + D * set + lane_base;
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
          uint32_t ov[32];
          tmem_ld32(my_o + 32 * cb, ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
          tmem_st32(my_o + 32 * cb, ov);
        }
        tmem_wait_st();
      }
      m_ref = m_new;
      const float ref = m_ref == -INFINITY ? 0.f : m_ref;
      if (m_l != m_ref) {  // the row sum follows the reference
        l_set *= ex2(m_l - m_ref);
        m_l = m_ref;
      }
      // P = exp2(x - ref) as hi (e4m3) + mid (e4m3) + lo (e5m2), four tokens to a column
      uint32_t ph[4 * kNp], pm[4 * kNp], pl[4 * kNp];
#pragma unroll
      for (int q = 0; q < kNp; ++q) {
        const uint64_t c2 = f32x2(__float_as_uint(cq[q]), __float_as_uint(cq[q]));
        const uint64_t nr2 = f32x2(__float_as_uint(aq[q] - ref), __float_as_uint(aq[q] - ref));
        uint64_t sum2 = 0ull;
#pragma unroll
        for (int j = 8 * q; j < 8 * q + 8; j += 2) {  // pairs j, j + 1 = four tokens = one column
          uint16_t hi[2], mid[2], lo[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const uint64_t x2 = fma_f32x2(f32x2(sv[2 * (j + e)], sv[2 * (j + e) + 1]), c2, nr2);
            float x0, x1;
            f32x2_split(x2, x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            sum2 = add_f32x2(sum2, f32x2(__float_as_uint(p0), __float_as_uint(p1)));
            split_e4m3_e4m3_e5m2_x2(p0, p1, hi[e], mid[e], lo[e]);
          }
          ph[j >> 1] = static_cast<uint32_t>(hi[0]) | (static_cast<uint32_t>(hi[1]) << 16);
          pm[j >> 1] = static_cast<uint32_t>(mid[0]) | (static_cast<uint32_t>(mid[1]) << 16);
          pl[j >> 1] = static_cast<uint32_t>(lo[0]) | (static_cast<uint32_t>(lo[1]) << 16);
        }
        float s0, s1;
        f32x2_split(sum2, s0, s1);
        l_set = fmaf(s0 + s1, iq[q], l_set);
      }
      if (it >= 2) {
        // (P goes over its own S; this wait keeps the set's view of the barrier one phase behind at most,
        // which the parity waits on it rely on)
        ok = mbar_spin_bounded(my_pv, (k - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
      }
      // columns 0..15 the high parts of the iteration's 64 tokens, 16..31 the middle parts, 32..47 the low
      // parts (the A operands of the three P . V products); half rows: the other 32 tokens' columns are zero
      if constexpr (kHalf) {
        const uint32_t zeros[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        const uint32_t mine = sp_buf + 8 * half, other = sp_buf + 8 * (half ^ 1);  // (warp-uniform)
        tmem_st8(mine, ph);       tmem_st8(other, zeros);
        tmem_st8(mine + 16, pm);  tmem_st8(other + 16, zeros);
        tmem_st8(mine + 32, pl);  tmem_st8(other + 32, zeros);
      } else {
        tmem_st16(sp_buf, ph);
        tmem_st16(sp_buf + 16, pm);
        tmem_st16(sp_buf + 32, pl);
      }
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_tc(my_p);
    }

    // ---- finalise: this set's last PV, then the merge of the accumulators that hold parts of a row: the
    // two sets' (and, with half rows, those of lanes r and r + 64)
    bool ok = alive;
    {
      const int last = n_iters - 1 - ((n_iters - 1 - set) & 1);  // this set's last iteration, if any
      if (alive && last >= set) {
        ok = mbar_wait_bounded(my_pv, (last >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
        tc_fence_after();
      }
      if (m_l != m_ref) l_set *= ex2(m_l - m_ref);
      m_sh[set * kTcRows + t] = m_ref;
      l_sh[set * kTcRows + t] = l_set;
    }
    // every softmax warp reaches this point together with its error view settled; all P . V have completed
    asm volatile("bar.sync 2, %0;" ::"n"(kTcSoftmaxWarps * 32) : "memory");
    const int dev_err = max(err, *cta_err);
    if (dev_err && tid == 0) report(p.status, dev_err);
    const bool valid_row = r < rows_total;
    const bool have = alive && ok && n_iters > 0 && *cta_err == 0;  // warp-uniform (and CTA-uniform: cta_err is settled)
    float l = 0.f, w0 = 0.f, w1 = 0.f;  // weights of this lane's two accumulators (one per set)
    if (have) {
      const float m0 = m_sh[t], m1 = m_sh[kTcRows + t];
      float M = fmaxf(m0, m1);
      const int tp = t ^ (kTcRows / 2);  // half rows: the lane that holds the row's other half
      if constexpr (kHalf) M = fmaxf(M, fmaxf(m_sh[tp], m_sh[kTcRows + tp]));
      auto wgt = [&](float m) { return m == -INFINITY ? 0.f : ex2(m - M); };
      w0 = wgt(m0);
      w1 = wgt(m1);
      l = w0 * l_sh[t] + w1 * l_sh[kTcRows + t];
      if constexpr (kHalf) l += wgt(m_sh[tp]) * l_sh[tp] + wgt(m_sh[kTcRows + tp]) * l_sh[kTcRows + tp];
      m_ref = M;
    }
    const bool live = !dev_err && have && l > 0.f;
    const float inv = live ? 1.f / l : 0.f;
    const int64_t qrow = (static_cast<int64_t>(b) * T + i_tok) * p.num_q_heads + g * G + (r % G);
    constexpr float kLn2 = 0.6931471805599453f;
    // set x handles columns [D/2 x, D/2 (x + 1)) of the row, 32 at a time: this lane's accumulators, weighted
    uint32_t ov[D / 64][32];
#pragma unroll
    for (int cc = 0; cc < D / 64; ++cc) {
      const int cb = (D / 64) * set + cc;
      if (have) {
        tmem_ld32(tmem_o + lane_base + 32 * cb, ov[cc]);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[cc][j] = __float_as_uint(__uint_as_float(ov[cc][j]) * w0);
        if (n_iters > 1) {  // (the second set's accumulator exists from two iterations on)
          uint32_t o1[32];
          tmem_ld32(tmem_o + D + lane_base + 32 * cb, o1);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            ov[cc][j] = __float_as_uint(fmaf(__uint_as_float(o1[j]), w1, __uint_as_float(ov[cc][j])));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[cc][j] = 0u;
      }
    }
    if constexpr (kHalf) {
      // lanes from 64 hand their part to the lane that stores the row, through the idle ring
      // ([column][row]: a warp's lanes write consecutive words)
      float* xch = reinterpret_cast<float*>(smem);
      if (half == 1) {
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc)
#pragma unroll
          for (int j = 0; j < 32; ++j)
            xch[(((D / 64) * set + cc) * 32 + j) * (kTcRows / 2) + (t & (kTcRows / 2 - 1))] = __uint_as_float(ov[cc][j]);
      }
      asm volatile("bar.sync 2, %0;" ::"n"(kTcSoftmaxWarps * 32) : "memory");
      if (half == 0) {
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc)
#pragma unroll
          for (int j = 0; j < 32; ++j)
            ov[cc][j] = __float_as_uint(__uint_as_float(ov[cc][j]) +
                                        xch[(((D / 64) * set + cc) * 32 + j) * (kTcRows / 2) + t]);
      }
    }
    if (valid_row && half == 0) {
#pragma unroll
      for (int cc = 0; cc < D / 64; ++cc) {
        const int cb = (D / 64) * set + cc;
        if (split) {
          float4* dst = reinterpret_cast<float4*>(p.part_o + (qrow * p.max_chunks + p.chunk_slot0 + c) * D + 32 * cb);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(__uint_as_float(ov[cc][4 * j]) * inv, __uint_as_float(ov[cc][4 * j + 1]) * inv,
                                 __uint_as_float(ov[cc][4 * j + 2]) * inv, __uint_as_float(ov[cc][4 * j + 3]) * inv);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(p.out + qrow * D + 32 * cb);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              w[e] = pack2<false>(__uint_as_float(ov[cc][8 * j + 2 * e]) * inv,
                                  __uint_as_float(ov[cc][8 * j + 2 * e + 1]) * inv);
            dst[j] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (split && set == 0)
        p.part_lse[qrow * p.max_chunks + p.chunk_slot0 + c] = live ? (m_ref + __log2f(l)) * kLn2 : -INFINITY;
    }
  };
  if constexpr (!kFp8) {
    load_q();
    if (warp == kTcProducerWarp) producer_role(); else wait_q();
    if (warp == kTcMmaWarp) s_issue_role();
    else if (warp == kTcPvWarp) pv_issue_role();
    else if (warp < kTcSoftmaxWarps) softmax_role();
  } else {
    // by warpgroup, each first taking or giving up registers (the setmaxnreg sits at the head of the code
    // that only that group runs)
    if (warp < kTcSoftmaxWarps) {
      reg_alloc_inc<kTcRegsSoftmax>();
      load_q();
      wait_q();
      if (half_rows) softmax_role_fp8(std::integral_constant<int, 2>{});
      else softmax_role_fp8(std::integral_constant<int, 4>{});
    } else {
      reg_alloc_dec<kTcRegsControl>();
      if (warp == kTcProducerWarp) {
        producer_role();
      } else {
        wait_q();
        if (warp == kTcMmaWarp) s_issue_role();
        else if (warp == kTcPvWarp) pv_issue_role();
      }
    }
  }

  // ---- teardown: everyone is done with tensor memory before it is released
  tc_fence_before();
  __syncthreads();
  if (warp == kTcMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

bool attention_mq_tc_supports(const MqParams& mp) {
  const AttnParams& p = mp.a;
  if (p.geom.dtype == PDA_BF16) {
    if (p.geom.head_dim != 128 && p.geom.head_dim != 64) return false;
  } else {
    if (p.geom.head_dim != 128 || p.k_scale == nullptr || p.v_scale == nullptr) return false;
  }
  if (p.group < 1 || mp.n_q < 1 || p.geom.num_pages < 1) return false;
  if (!(p.scale > 0.f) || !(p.scale < INFINITY)) return false;  // the row maximum is taken before scaling
  const int64_t rows = static_cast<int64_t>(mp.n_q) * p.group;
  return p.geom.num_kv_heads * ((rows + kTcRows - 1) / kTcRows) <= 65535;
}

namespace {
template <int D, bool kFp8>
cudaError_t launch_tc(const CUtensorMap& k_map, const CUtensorMap& v_map, const MqParams& mp, cudaStream_t stream) {
  const AttnParams& p = mp.a;
  using C = TcCfg<D, kFp8>;
  cudaError_t e = cudaFuncSetAttribute(attention_mq_tc_kernel<D, kFp8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int rows_total = mp.n_q * p.group;
  const int n_rb = (rows_total + kTcRows - 1) / kTcRows;
  const unsigned chunks = p.chunk_tokens > 0 ? static_cast<unsigned>(mp.n_chunks_grid) : 1u;
  dim3 grid(chunks, p.geom.num_kv_heads * n_rb, p.batch);
  attention_mq_tc_kernel<D, kFp8><<<grid, C::kThreads, C::kSmemBytes, stream>>>(k_map, v_map, mp);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_attention_mq_tc(const MqParams& mp, cudaStream_t stream) {
  const AttnParams& p = mp.a;
  const bool fp8 = p.geom.dtype != PDA_BF16;
  const int eb = fp8 ? 1 : 2;
  alignas(64) CUtensorMap k_map, v_map;
  // K is copied one 128-byte line of its rows at a time (so that the pages of an iteration stack), V as whole tiles
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb, /*box_lines=*/1) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb))
    return cudaErrorNotSupported;
  if (fp8) return launch_tc<128, true>(k_map, v_map, mp, stream);
  return p.geom.head_dim == 128 ? launch_tc<128, false>(k_map, v_map, mp, stream)
                                : launch_tc<64, false>(k_map, v_map, mp, stream);
}

}  // namespace pda
