// Multi-query paged attention on the 5th-generation tensor cores (tcgen05 + TMEM): verification of a
// block of draft tokens, and the shared-prefix part of a decode batch; same contract as attention_mq.cu.
// Up to 128 query rows (query tokens x group size) per CTA against one sequence's pages. bf16 KV with
// head_dim 128 or 64 (the figures in this comment are for 128), or e4m3 KV with head_dim 128.
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
//               (bar_sfree) -> commit(bar_s[j&1])
//   PV warp:    wait bar_p[i&1] -> PV(i), l(i) -> commit(stage empty), commit(bar_pv[i&1])
//   softmax:    wait bar_s[i&1] -> tcgen05.ld S -> arrive(bar_sfree) -> mask (boundary tiles), row max
//               of the raw scores -> running max of iteration i-1 from the other set (bar_m, shared
//               memory) -> publish the new one -> (rarely, after waiting for PV(i-1)) rescale O and l in
//               TMEM when the max grew by more than 2^8 -> wait PV(i-2) (P buffer free) -> P =
//               exp2(S * scale - ref) as bf16 pairs (packed f32x2 FMA, one exp2 per element) ->
//               tcgen05.st P -> arrive(bar_p[i&1])
// e4m3 KV: the tensor core has no bf16 x e4m3 mode and e4m3 x e4m3 would quantise Q and P, so the tiles
// are converted. The TMA ring holds the raw tiles (128-byte rows), four converter warps (8-11) write
// each iteration's K and V as an f16 operand block (exact conversion, the page's scale folded in, rows
// past the sequence end zeroed) into one of three conversion slots, and Q, P and the tile of ones are
// f16 as well. That variant runs 16 warps (producer 12, S issue 13, PV issue 14) as four warpgroups and
// moves registers from the converter and control groups to the softmax groups (setmaxnreg).
// All mbarrier waits are bounded; TMEM is always released before the CTA exits.
#include "common.cuh"
#include "tma_ptx.cuh"

namespace pda {

namespace {

constexpr int kTcRows = 128;            // query rows per CTA (UMMA M)
constexpr int kTcPagesPerIter = 4;      // 64 tokens per iteration
constexpr int kTcOnesBytes = 2048;                         // bf16 ones: B operand [16 tokens][16 columns] of the row-sum MMA
constexpr int kTcMBytes = 2 * kTcRows * 4;                 // running row maxima handed between the two softmax sets
// Sizes that depend on head_dim D (128 or 64) and on the cache's element type. A 16-bit row is D / 64
// lines of 128 bytes. An operand block = what the tensor core reads for one iteration: K of 4 pages as
// [lines][64 tokens][128 B], then 4 V page tiles. bf16 caches: the TMA ring holds operand blocks. e4m3
// caches (D = 128): the ring holds the raw tiles (128-byte rows) and four converter warps turn them into
// f16 operand blocks, exactly and with the page's scales folded in, in kConvSlots conversion slots.
template <int D, bool kFp8>
struct TcCfg {
  static_assert(!kFp8 || D == 128, "e4m3 is built for head_dim 128");
  static constexpr int kLines = D / 64;
  static constexpr int kTileBytes = kPageSize * D * 2;          // one 16-bit K or V page tile: 4096 / 2048
  static constexpr int kKBytes = kTcPagesPerIter * kTileBytes;  // K of 4 pages as [lines][64 tokens][128 B]
  static constexpr int kOperandBytes = 2 * kKBytes;             // K block, then 4 V page tiles: 32 / 16 KB
  static constexpr int kRawTileBytes = kPageSize * D;           // one e4m3 page tile: 2048
  static constexpr int kStageBytes = kFp8 ? 2 * kTcPagesPerIter * kRawTileBytes : kOperandBytes;
  static constexpr int kStages = kFp8 ? 6 : 6 * 128 / D;        // 192 KB of ring for 16-bit caches, 96 KB for e4m3
  // (a slot is free again after the PV that read it; four slots with four raw stages, and separate pools
  // for K and V, were measured no faster: the converters' instructions share the schedulers with the
  // softmax warps, which is what stretches an iteration from 0.72 to 1.0 us)
  static constexpr int kConvSlots = kFp8 ? 3 : 0;
  static constexpr int kScaleBytes = kFp8 ? kStages * 2 * kTcPagesPerIter * 4 : 0;  // per stage: 4 K and 4 V scales
  static constexpr int kSmemBytes = kStages * kStageBytes + kConvSlots * kOperandBytes + kTcOnesBytes + kTcMBytes +
                                    kScaleBytes + 512 + 1024;
  // warps: softmax 0-7; then (e4m3: converters 8-11) producer, S issue (+ TMEM allocation), PV issue
  static constexpr int kProducerWarp = kFp8 ? 12 : 8, kMmaWarp = kProducerWarp + 1, kPvWarp = kProducerWarp + 2;
  static constexpr int kThreads = kFp8 ? 512 : 352;
};
constexpr int kTcSoftmaxWarps = 8;      // two sets of 4: set x takes the iterations it with it % 2 == x
// e4m3 variant: four warpgroups whose registers are redistributed at the start (setmaxnreg):
// 2 x 128 x 176 (softmax) + 128 x 80 (converters) + 128 x 64 (producer, issuers, one spare warp) <= 65536
constexpr uint32_t kTcRegsSoftmax = 176, kTcRegsConvert = 80, kTcRegsControl = 64;
// Tensor memory columns (32-bit each, 128 lanes = query rows): S buffers 0..63 and 64..127 (f32),
// O 128..255 (f32), Q 256..319 (bf16 pairs along d), P buffers 320..351 and 352..383 (bf16 pairs
// along tokens). Allocations are powers of two.
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = 128, kTmemQ = 256, kTmemP = 320, kTmemL = 384;  // l: row sums of P, 16 columns (all equal)
constexpr float kRescaleThreshold = 8.f;  // log2 units: O is rescaled only when the max grows this much

// Spinning bounded wait (no suspension): the waits on the MMA/softmax hand-off are short and on the
// critical path, where the wake-up latency of a suspended try_wait shows.
__device__ __forceinline__ bool mbar_spin_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 24); ++i)
    if (mbar_test_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void mbar_arrive_tc(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[tmem] . B[smem descriptor]; accumulate == 0 overwrites D. A is read from tensor memory
// (lane = row, 32-bit column = two consecutive k elements).
__device__ __forceinline__ void tc_mma_ts_if(uint32_t leader, uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred pe, pa;\n\tsetp.ne.b32 pe, %5, 0;\n\tsetp.ne.b32 pa, %4, 0;\n\t"
      "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pa;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}
__device__ __forceinline__ void tc_commit_if(uint32_t leader, uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred pe;\n\tsetp.ne.b32 pe, %1, 0;\n\t"
      "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar), "r"(leader) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 version field.
__device__ __forceinline__ uint64_t tc_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu) |
         (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: f32 accumulate, A and B both bf16 or both f16, A K-major, M = 128.
__host__ __device__ constexpr uint32_t tc_idesc(int n, bool b_mn_major, bool f16) {
  return (1u << 4) | ((f16 ? 0u : 1u) << 7) | ((f16 ? 0u : 1u) << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTcRows >> 4) << 24);
}
template <uint32_t kRegs>
__device__ __forceinline__ void reg_alloc_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegs)); }
template <uint32_t kRegs>
__device__ __forceinline__ void reg_alloc_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegs)); }
// 16 e4m3 values (one 16-byte chunk) -> 16 f16 values times a scale, as two 16-byte chunks
__device__ __forceinline__ void e4m3x16_to_f16(const uint4& in, uint32_t scale2, uint4& lo, uint4& hi) {
  auto cv = [&](uint32_t w, uint32_t& a, uint32_t& b) {
    a = e4m3x2_to_f16x2(w & 0xffffu);
    b = e4m3x2_to_f16x2(w >> 16);
    asm("mul.rn.f16x2 %0, %0, %1;" : "+r"(a) : "r"(scale2));
    asm("mul.rn.f16x2 %0, %0, %1;" : "+r"(b) : "r"(scale2));
  };
  cv(in.x, lo.x, lo.y); cv(in.y, lo.z, lo.w); cv(in.z, hi.x, hi.y); cv(in.w, hi.z, hi.w);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// Packed pairs of f32 (sm_100): one instruction per two elements in the softmax inner loops.
__device__ __forceinline__ uint64_t f32x2(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

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
  uint8_t* conv_smem = smem + kTcStages * kTcStageBytes;             // e4m3: kConvSlots operand blocks
  uint8_t* ones_smem = conv_smem + C::kConvSlots * C::kOperandBytes;
  float* m_sh = reinterpret_cast<float*>(ones_smem + kTcOnesBytes);        // [2][128]
  float* scale_sh = m_sh + 2 * kTcRows;                                    // e4m3: [stage][4 K scales, 4 V scales]
  // full[], empty[], s[2], p[2], pv[2], sfree[2], m[2], conv_full[4], conv_free[4]
  uint64_t* bars = reinterpret_cast<uint64_t*>(ones_smem + kTcOnesBytes + kTcMBytes + C::kScaleBytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kTcStages + 18);
  int* cta_err = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.group, T = mp.n_q;
  const int rows_total = T * G;
  const int n_rb = (rows_total + kTcRows - 1) / kTcRows;
  const int c = blockIdx.x, g = blockIdx.y / n_rb, rb = blockIdx.y % n_rb;
  const bool split = p.chunk_tokens > 0;
  int b = blockIdx.z;
  if (!split && mp.kv_len_fixed == 0 && p.batch > 1 && p.batch <= 128) {  // (ranking costs O(batch^2/threads))
    // unsplit units differ in length: the CTA with blockIdx.z = r serves the r-th longest sequence
    int* lens = reinterpret_cast<int*>(smem);
    for (int j = tid; j < p.batch; j += kTcThreads) lens[j] = max(p.seq_lens[j], 0);
    __syncthreads();
    for (int j = tid; j < p.batch; j += kTcThreads) {
      const int Lj = lens[j];
      int rank = 0;
      for (int i = 0; i < p.batch; ++i) rank += (lens[i] > Lj) || (lens[i] == Lj && i < j);
      if (rank == static_cast<int>(blockIdx.z)) *cta_err = j;
    }
    __syncthreads();
    b = *cta_err;
    __syncthreads();  // lens aliases the ring and cta_err is reused below
  }

  const int L = mp.kv_len_fixed > 0 ? mp.kv_len_fixed : max(p.seq_lens[b], 0);
  int t0 = p.first_token, t1 = L;
  if (split) {
    t0 = p.first_token + c * p.chunk_tokens;
    if (t0 >= L) return;
    t1 = min(t0 + p.chunk_tokens, L);
  }
  // once any CTA of this launch has reported a timed-out wait, the rest do not start
  if (p.status != nullptr && *reinterpret_cast<volatile int32_t*>(p.status) == PDA_DEV_TIMEOUT) return;
  int err = 0;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ||
      (split && static_cast<int64_t>(L - p.first_token) >
                    static_cast<int64_t>(p.max_chunks - p.chunk_slot0) * p.chunk_tokens))
    err = PDA_DEV_BAD_SEQ_LEN;
  const int page0 = t0 / kPageSize;
  const int n_pages = err ? 0 : (t1 + kPageSize - 1) / kPageSize - page0;
  const int n_iters = (n_pages + kTcPagesPerIter - 1) / kTcPagesPerIter;

  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kTcStages;
  const uint32_t bar_s = empty0 + 8 * kTcStages, bar_p = bar_s + 16, bar_pv = bar_p + 16;  // two of each
  const uint32_t bar_sfree = bar_pv + 16, bar_m = bar_sfree + 16;
  const uint32_t conv_full0 = bar_m + 16, conv_free0 = conv_full0 + 32;  // four of each (e4m3)
  for (int i = tid; i < kTcOnesBytes / 4; i += kTcThreads)
    reinterpret_cast<uint32_t*>(ones_smem)[i] = kFp8 ? 0x3C003C00u : 0x3F803F80u;  // 1.0 as f16 / bf16 pairs
  fence_proxy_async();  // read by the tensor core through the async proxy
  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kFp8 ? 4 : 1);  // released by the PV MMAs' commit, or by the 4 converter warps
    }
    for (int k = 0; k < 4; ++k) {
      mbar_init(conv_full0 + 8 * k, 4);  // an operand block converted (4 converter warps)
      mbar_init(conv_free0 + 8 * k, 1);  // the PV MMAs that read it have completed
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(bar_s + 8 * k, 1);
      mbar_init(bar_p + 8 * k, 4);   // one arrival per warp of the softmax set that owns the iteration
      mbar_init(bar_pv + 8 * k, 1);
      mbar_init(bar_sfree + 8 * k, 4);
      mbar_init(bar_m + 8 * k, 4);
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

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + kTmemO;  // S buffer k at tmem_s + 64 k
  const uint32_t tmem_q = tmem_base + kTmemQ, tmem_p = tmem_base + kTmemP;  // P buffer k at tmem_p + 32 k

  const int32_t* table = p.block_table + static_cast<int64_t>(b) * p.block_table_stride;

  // The roles, as closures: the two variants dispatch them differently (the e4m3 one by warpgroup, each
  // group first taking or giving up registers).
  // ---- Q: row r -> (query token r / G, head r % G) goes to TMEM lane r as the A operand of S = Q . K^T
  auto load_q = [&]() {
    if (warp < 4) {
      const int r = rb * kTcRows + tid;
      const bool valid = r < rows_total;
      const int64_t qrow = (static_cast<int64_t>(b) * T + r / G) * p.num_q_heads + g * G + (r % G);
      const uint4* src = reinterpret_cast<const uint4*>(p.q + qrow * D);
  #pragma unroll
      for (int h = 0; h < D / 64; ++h) {  // 64 bf16 = 32 columns per store
        uint32_t qv[32];
  #pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          const uint4 v = valid ? src[h * 8 + ch] : make_uint4(0u, 0u, 0u, 0u);
          qv[4 * ch] = v.x; qv[4 * ch + 1] = v.y; qv[4 * ch + 2] = v.z; qv[4 * ch + 3] = v.w;
          if (kFp8) {  // the e4m3 variant multiplies in f16: bf16 pairs -> f16 pairs
  #pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t w = qv[4 * ch + e];
              qv[4 * ch + e] = pack2<true>(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
            }
          }
        }
        tmem_st32(tmem_q + (static_cast<uint32_t>(warp * 32) << 16) + 32 * h, qv);
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
    float ks = 0.f, vs = 0.f;  // e4m3: the page's dequantisation factors
    for (int it = 0; it < u_iters; ++it) {
      const int s = it % kTcStages;
      if ((it & 7) == 0) {  // page ids of the next 8 iterations (32 pages), one per lane
        pg = 0;
        if (it * kTcPagesPerIter + lane < u_pages) {
          const int v = table[page0 + it * kTcPagesPerIter + lane];
          pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
          if (kFp8) {
            ks = p.k_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g];
            vs = p.v_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g];
          }
        }
      }
      bool ok = true;
      if (it >= kTcStages) ok = mbar_wait_bounded(empty0 + 8 * s, ((it / kTcStages) - 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); break; }
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      const uint32_t stage = ring + s * kTcStageBytes, bar = full0 + 8 * s;
      if (kFp8) {  // this stage's scales, written by the lanes that hold its pages (seen through the full barrier)
        if ((lane >> 2) == (it & 7)) {
          scale_sh[s * 8 + (lane & 3)] = ks;
          scale_sh[s * 8 + 4 + (lane & 3)] = vs;
        }
        __syncwarp();
      }
      mbar_expect_tx_if(leader, bar, n_here * 2 * (kFp8 ? C::kRawTileBytes : kTcTileBytes));
      // K: one copy per 128-byte line so that page j's 16 rows follow page j-1's in each line block
      // (an e4m3 row is one line; raw V tiles follow the raw K block)
      auto load_page = [&](int j) {
        const int page_raw = __shfl_sync(0xffffffffu, pg, (it & 7) * kTcPagesPerIter + j);
        bad |= page_raw < 0;
        const int page = max(page_raw, 0);
        if (kFp8) {
          tma_load_5d_if(leader, stage + j * C::kRawTileBytes, &k_map, bar, 0, g, page);
          tma_load_5d_if(leader, stage + (kTcPagesPerIter + j) * C::kRawTileBytes, &v_map, bar, 0, g, page);
        } else {
#pragma unroll
          for (int ln = 0; ln < C::kLines; ++ln)
            tma_load_5d_if(leader, stage + ln * (kTcKBytes / C::kLines) + j * (kPageSize * 128), &k_map, bar, ln, g, page);
          tma_load_5d_if(leader, stage + kTcKBytes + j * kTcTileBytes, &v_map, bar, 0, g, page);
        }
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
    constexpr uint32_t idesc_s = tc_idesc(kTcPagesPerIter * kPageSize, false, kFp8);
    const uint32_t leader = elect_one();
    // warp-uniform copies (a shuffle from lane 0 tells the compiler so)
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    const int u_iters = __shfl_sync(0xffffffffu, n_iters, 0);
    const int u_pages = __shfl_sync(0xffffffffu, n_pages, 0);
    const int u_tail0 = __shfl_sync(0xffffffffu, L - page0 * kPageSize, 0);  // tokens from the first page to the end
    bool ok = true;
    // the iteration's operand block: its ring stage (16-bit caches) or conversion slot (e4m3), and the
    // phase parity of that block's "ready" barrier
    constexpr uint32_t kBlocks = kFp8 ? C::kConvSlots : kTcStages;
    const uint32_t blocks0 = kFp8 ? smem_u32(conv_smem) : ring;
    const uint32_t ready0 = kFp8 ? conv_full0 : full0;
    uint32_t stage_i = 0, stage_par = 0;
    for (int it = 0; it < u_iters; ++it) {
      // S(it) overwrites the buffer of S(it-2): the softmax warps have loaded that into registers
      if (it >= 2) ok = mbar_wait_bounded(bar_sfree + 8 * (it & 1), ((it - 2) >> 1) & 1);
      if (ok) ok = mbar_wait_bounded(ready0 + 8 * stage_i, stage_par);  // the block has landed / been converted
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t stage = blocks0 + stage_i * C::kOperandBytes;
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      const int tail = u_tail0 - (it * kTcPagesPerIter + n_here - 1) * kPageSize;  // valid rows of the last page here
      if (!kFp8 && tail < kPageSize) {  // clear the rows past the sequence end in V (P is 0 there, V must be
                                        // finite); the e4m3 converters do it as they write the block
        const uint32_t vt = stage + kTcKBytes + (n_here - 1) * kTcTileBytes;
        constexpr int kChunksPerRow = D / 8;  // 16-byte chunks of a row
        for (int i = lane; i < (kPageSize - tail) * kChunksPerRow; i += 32) {
          const int r = tail + i / kChunksPerRow, ch = i % kChunksPerRow;
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_off(r, ch)), "r"(0));
        }
        fence_proxy_async();
        __syncwarp();
      }
      tc_fence_after();
      const uint32_t d = u_tmem + 64 * (it & 1);
      // S[:, 0..64) = Q . K^T over the 64 stacked token rows, contraction over d in 8 steps of 16
      // (rows of pages that were not loaded hold stale data: those columns are masked later)
      const uint64_t kd0 = tc_desc(stage, 16, 1024);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        // descriptor start addresses are in 16-byte units: +2 per k-step, next line block further on
        const uint64_t bd = kd0 + static_cast<uint64_t>((ks >> 2) * (kTcKBytes / C::kLines / 16) + (ks & 3) * 2);
        tc_mma_ts_if(leader, d, u_tmem + kTmemQ + 8 * ks, bd, idesc_s, ks > 0 ? 1u : 0u);
      }
      tc_commit_if(leader, bar_s + 8 * (it & 1));
      if (++stage_i == kBlocks) { stage_i = 0; stage_par ^= 1; }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };
  auto pv_issue_role = [&]() {
    // ================= PV issue: O += P . V and l += P . 1 =================
    constexpr uint32_t idesc_pv = tc_idesc(D, true, kFp8);
    constexpr uint32_t idesc_l = tc_idesc(16, false, kFp8);
    const uint64_t ones_desc = tc_desc(smem_u32(ones_smem), 16, 1024);
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    const int u_iters = __shfl_sync(0xffffffffu, n_iters, 0);
    const int u_pages = __shfl_sync(0xffffffffu, n_pages, 0);
    bool ok = true;
    constexpr uint32_t kBlocks = kFp8 ? C::kConvSlots : kTcStages;
    const uint32_t blocks0 = kFp8 ? smem_u32(conv_smem) : ring;
    uint32_t stage_i = 0;  // the iteration's operand block: ring stage or conversion slot
    for (int it = 0; it < u_iters; ++it) {
      ok = mbar_wait_bounded(bar_p + 8 * (it & 1), (it >> 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t stage = blocks0 + stage_i * C::kOperandBytes;
      const int n_here = min(kTcPagesPerIter, u_pages - it * kTcPagesPerIter);
      // O += P[:, 16j .. 16j+16) . V_j : one K = 16 step per page, V read MN-major
      const uint32_t pa0 = u_tmem + kTmemP + 32 * (it & 1);
      const uint64_t vd0 = tc_desc(stage + kTcKBytes, kPageSize * 128, 1024);  // LBO: next 64 columns of d, SBO: next 8 tokens
      // and l += P[:, 16j .. 16j+16) . 1 : the row sums of exactly the P that multiplies V
      auto pv_page = [&](int j) {
        const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
        tc_mma_ts_if(leader, u_tmem + kTmemO, pa0 + 8 * j, vd0 + static_cast<uint64_t>(j * (kTcTileBytes / 16)), idesc_pv, acc);
        tc_mma_ts_if(leader, u_tmem + kTmemL, pa0 + 8 * j, ones_desc, idesc_l, acc);
      };
      if (n_here == kTcPagesPerIter) {
#pragma unroll
        for (int j = 0; j < kTcPagesPerIter; ++j) pv_page(j);
      } else {
        for (int j = 0; j < n_here; ++j) pv_page(j);
      }
      // the stage may be refilled (the conversion slot rewritten) once these MMAs have read it
      tc_commit_if(leader, (kFp8 ? conv_free0 : empty0) + 8 * stage_i);
      tc_commit_if(leader, bar_pv + 8 * (it & 1));    // O and l updated, P buffer free again
      if (++stage_i == kBlocks) stage_i = 0;
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };
  auto convert_role = [&]() {
    if constexpr (kFp8) {
      // ================= e4m3 -> f16 converters: raw stage -> operand block in a conversion slot ==========
      // cvt.rn.f16x2.e4m3x2 is exact, the page's scale is folded in (one f16 multiply), rows past the
      // sequence end become zeros. A thread moves 4 K and 4 V chunks of 16 bytes per iteration (one of each
      // per page): raw row, chunk c (swizzled by the row) -> 16-bit row, chunks 2 (c % 4), 2 (c % 4) + 1 of
      // line c / 4.
      const int ct = tid - kTcSoftmaxWarps * 32;  // 0..127
      const uint32_t conv0 = smem_u32(conv_smem);
      // This thread's four chunks never change: chunk q of its four is row r = 16 q + ct / 8 (page q of the
      // iteration, slot ct / 8), raw chunk c = ct % 8. Offsets inside a raw half-stage / an operand block:
      const int rr = ct >> 3, c = ct & 7, sw = rr & 7;
      const uint32_t src_off = static_cast<uint32_t>(rr * 128 + ((c ^ sw) << 4));          // + q * raw tile
      const int line = c >> 2, c2 = (c & 3) * 2;
      const uint32_t k_off = static_cast<uint32_t>(line * (64 * 128) + rr * 128);           // + q * 16 rows
      const uint32_t v_off = static_cast<uint32_t>(kTcKBytes + line * (kPageSize * 128) + rr * 128);  // + q * V tile
      const uint32_t ch0 = static_cast<uint32_t>((c2 ^ sw) << 4), ch1 = static_cast<uint32_t>(((c2 + 1) ^ sw) << 4);
      uint32_t slot = 0, slot_par = 0, stage_i = 0, stage_par = 0;
      bool ok = true;
      for (int it = 0; it < n_iters; ++it) {
        ok = mbar_wait_bounded(full0 + 8 * stage_i, stage_par);                        // raw tiles have landed
        if (ok && it >= C::kConvSlots) ok = mbar_wait_bounded(conv_free0 + 8 * slot, slot_par ^ 1);  // PV(it - kConvSlots) done
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t raw = ring + stage_i * kTcStageBytes;
        const uint32_t dst = conv0 + slot * C::kOperandBytes;
        const float* sc = scale_sh + stage_i * 8;
        const int n_here = min(kTcPagesPerIter, n_pages - it * kTcPagesPerIter);
        const int valid_rows = min(L - (page0 + it * kTcPagesPerIter) * kPageSize, n_here * kPageSize);  // token rows of this block
#pragma unroll
        for (int q = 0; q < kTcPagesPerIter; ++q) {
          if (q < n_here) {  // (uniform)
            uint4 kin, vin, klo, khi, vlo, vhi;
            const uint32_t src = raw + q * C::kRawTileBytes + src_off;
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(kin.x), "=r"(kin.y), "=r"(kin.z), "=r"(kin.w) : "r"(src));
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(vin.x), "=r"(vin.y), "=r"(vin.z), "=r"(vin.w)
                         : "r"(src + kTcPagesPerIter * C::kRawTileBytes));
            e4m3x16_to_f16(kin, pack2<true>(sc[q], sc[q]), klo, khi);
            e4m3x16_to_f16(vin, pack2<true>(sc[4 + q], sc[4 + q]), vlo, vhi);
            if (q * kPageSize + rr >= valid_rows) {  // a row past the end of the sequence (last block only)
              klo = make_uint4(0u, 0u, 0u, 0u); khi = klo; vlo = klo; vhi = klo;
            }
            const uint32_t kd = dst + k_off + q * (kPageSize * 128), vd = dst + v_off + q * kTcTileBytes;
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(kd + ch0), "r"(klo.x), "r"(klo.y), "r"(klo.z), "r"(klo.w));
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(kd + ch1), "r"(khi.x), "r"(khi.y), "r"(khi.z), "r"(khi.w));
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(vd + ch0), "r"(vlo.x), "r"(vlo.y), "r"(vlo.z), "r"(vlo.w));
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(vd + ch1), "r"(vhi.x), "r"(vhi.y), "r"(vhi.z), "r"(vhi.w));
          }
        }
        fence_proxy_async();   // the tensor core reads the block through the async proxy
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_tc(conv_full0 + 8 * slot);   // block ready for S and PV
          mbar_arrive_tc(empty0 + 8 * stage_i);    // raw stage may be refilled
        }
        if (++slot == C::kConvSlots) { slot = 0; slot_par ^= 1; }
        if (++stage_i == kTcStages) { stage_i = 0; stage_par ^= 1; }
      }
      if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
    }
  };
  auto softmax_role = [&]() {
    // ================= softmax: TMEM lane t <-> query row t; set x takes iterations x, x+2, ... ==========
    // Two warps per scheduler, one of each set: while one waits (for S, for the other set's row maximum,
    // for its tcgen05.ld/st) the other keeps the exp2 unit busy, which is what bounds this part.
    const int set = warp >> 2, t = tid & (kTcRows - 1);
    const int r = rb * kTcRows + t;
    const int i_tok = r / G;
    const int lim = mp.causal ? min(L, L - T + i_tok + 1) : L;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;  // this warp's TMEM lanes
    const float scale_log2 = p.scale * 1.4426950408889634f;
    const uint32_t my_s = bar_s + 8 * set, my_p = bar_p + 8 * set, my_pv = bar_pv + 8 * set;
    const uint32_t my_sfree = bar_sfree + 8 * set, my_m = bar_m + 8 * set, other_m = bar_m + 8 * (set ^ 1);
    float m_ref = -INFINITY;   // reference max the accumulated O and l (both in tensor memory) are scaled by
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
        for (int j = 0; j < 32; ++j) mxs[j & 3] = fmaxf(mxs[j & 3], __uint_as_float(sv[h][j]));
      const float mx = fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])) * scale_log2;
      // the reference after iteration it-1 comes from the other set
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
      if (it >= 2) {  // PV(it-2) has finished reading the P buffer this iteration writes
        ok = mbar_spin_bounded(my_pv, (k - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
      }
      if (it > 0 && __any_sync(0xffffffffu, need)) {
        // O and l may only be touched once PV(it-1) has completed; PV(it) is not issued before this
        // warp arrives on bar_p below, and the other set rescales only after PV(it)
        ok = mbar_spin_bounded(bar_pv + 8 * (set ^ 1), ((it - 1) >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        const float alpha = need ? ex2(m_ref - m_new) : 1.f;
#pragma unroll
        for (int cb = 0; cb < D / 32 + 1; ++cb) {  // O, then the block of columns that holds l
          uint32_t ov[32];
          tmem_ld32(tmem_o + lane_base + (cb < D / 32 ? 32 * cb : kTmemL - kTmemO), ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
          tmem_st32(tmem_o + lane_base + (cb < D / 32 ? 32 * cb : kTmemL - kTmemO), ov);
        }
        tmem_wait_st();
      }
      m_ref = m_new;
      const float ref = m_ref == -INFINITY ? 0.f : m_ref;
      // P = exp2(S * scale_log2 - ref) as bf16 pairs into TMEM lane t: the A operand of O += P . V
      // (one packed FMA per two elements; masked columns stay -inf -> 0)
      const uint64_t c2 = f32x2(__float_as_uint(scale_log2), __float_as_uint(scale_log2));
      const uint64_t nr2 = f32x2(__float_as_uint(-ref), __float_as_uint(-ref));
      uint32_t pw[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const uint64_t x2 = fma_f32x2(f32x2(sv[j >> 4][(2 * j) & 31], sv[j >> 4][(2 * j + 1) & 31]), c2, nr2);
        float x0, x1;
        f32x2_split(x2, x0, x1);
        pw[j] = pack2<kFp8>(ex2(x0), ex2(x1));  // (f16 pairs in the e4m3 variant, bf16 otherwise)
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
        ok = mbar_spin_bounded(bar_m + 8 * (last & 1), (last >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) m_ref = m_sh[(last & 1) * kTcRows + t];
      }
      if (ok) {
        ok = mbar_wait_bounded(bar_pv + 8 * (last & 1), (last >> 1) & 1);
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
  if constexpr (!kFp8) {
    load_q();
    if (warp == kTcProducerWarp) producer_role(); else wait_q();
    if (warp == kTcMmaWarp) s_issue_role();
    else if (warp == kTcPvWarp) pv_issue_role();
    else if (warp < kTcSoftmaxWarps) softmax_role();
  } else {
    // four warpgroups; registers go from the converter and control warps to the softmax warps (each group
    // executes its setmaxnreg at the head of the code that only it runs)
    if (warp < kTcSoftmaxWarps) {
      reg_alloc_inc<kTcRegsSoftmax>();
      load_q();
      wait_q();
      softmax_role();
    } else if (warp < kTcSoftmaxWarps + 4) {
      reg_alloc_dec<kTcRegsConvert>();
      wait_q();
      convert_role();
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
