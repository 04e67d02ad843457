// Multi-query paged attention over e4m3 caches on tcgen05 + TMEM, persistent CTAs: the tiles and the
// arithmetic of the e4m3 path of attention_mq_tc.cu (e4m3 x e4m3 products on the cache's bytes, Q as two
// and the softmax weights as three 8-bit parts, page scales through the softmax, one accumulator per
// softmax set, rows held twice when there are at most 64), for unsplit calls, with one CTA per SM walking
// through many (sequence, kv head, row block) units instead of one CTA per unit.
// Measured on the one-unit kernel (16 draft tokens, shared-prefix e4m3 batch, 58 k clocks per unit): 4.6 k
// clocks from entry to the set-up barrier, 7.6 k for loading Q and splitting it into e4m3 parts, 3 k to the
// first P, and 5 k from the last P to the stored output -- a third of the unit, during which the SM
// fetches nothing. Here
//   - barriers, tensor memory and the order of the sequences are set up once per CTA;
//   - the TMA producer runs on into the next unit's tiles while the current unit drains;
//   - a warp of its own (the stager) loads and splits the NEXT unit's Q rows into shared memory while the
//     current unit runs; at the boundary the softmax warps only copy them to tensor memory;
//   - nothing waits on a CTA-wide barrier between units: the hand-overs are mbarriers (Q staged, stage
//     free, Q in tensor memory), and iterations are numbered through all units of a CTA (gi), with ring
//     stages, S/P buffers, softmax sets and barrier phases following gi.
// Units are ordered by the length of their sequence (longest first) and dealt to the CTAs in serpentine
// order. All mbarrier waits are bounded; tensor memory is released before the CTA exits.
#include <type_traits>

#include "common.cuh"
#include "tma_ptx.cuh"
#include "tcgen05_ptx.cuh"

namespace pda {

namespace {

constexpr int kERows = kUmmaRows;                     // query rows per unit (UMMA M)
constexpr int kED = 128;
constexpr int kEPagesPerIter = 4;                     // 64 tokens per iteration
constexpr int kETileBytes = kPageSize * kED;          // one K or V page tile: 2048
constexpr int kEKBytes = kEPagesPerIter * kETileBytes;  // K of 4 pages: [64 tokens][128 B]
constexpr int kEStageBytes = 2 * kEKBytes;            // K block, then 4 V page tiles: 16 KB
constexpr int kEStages = 11;
constexpr int kEQPitch = 272;                         // staged Q row: 128 B high parts | 128 B low parts | 16 B pad, so that
                                                      // a warp's 16-byte accesses to 32 rows spread over all banks
constexpr int kEQxBytes = kERows * kEQPitch;          // the stage; half rows: 64 rows of it, then an area of the same size
                                                      // for the exchange between lanes r + 64 and r and for the output rows
constexpr int kEMaxBatch = 1024;                      // lengths and order of the sequences in shared memory
constexpr int kEBars = 2 * kEStages + 3 + 2 + 2 + 3 + 3;  // full, empty, s3, p, pv, buf, q / qfull / qfree
constexpr int kESmemBytes = kEStages * kEStageBytes + kEQxBytes + 2 * kERows * 4 /* m */ + 2 * kERows * 4 /* l */ +
                            kERows * 4 /* row constants */ + kEStages * 16 * 4 /* page constants */ +
                            kEMaxBatch * 4 + kEMaxBatch * 2 + kEBars * 8 + 64 + 1024;
constexpr int kESoftmaxWarps = 8, kEProducerWarp = 8, kEMmaWarp = 9, kEPvWarp = 10, kEStagerWarp = 11;
constexpr int kEThreads = 384;
constexpr uint32_t kERegsSoftmax = 208, kERegsControl = 72;
// Tensor memory columns: three S / P buffers 0..63, 64..127, 128..191 (iteration gi uses gi % 3), the two
// sets' accumulators 192..319 and 320..447, Q 448..511 (32 columns of high parts, 32 of low parts).
constexpr uint32_t kETmemCols = 512, kETmemO = 192, kETmemQ = 448;
constexpr int kEBufs = 3;
constexpr float kERescaleThreshold = 8.f;
constexpr float kERefBelowMax = 4.f;

struct EUnit {
  int b, g, rb;      // sequence, kv head, block of 128 query rows
  int L, err;        // length; PDA_DEV_BAD_SEQ_LEN when the table cannot describe it
  int n_pages, n_iters;
};

__global__ void __launch_bounds__(kEThreads, 1)
attention_mq_tc8p_kernel(const __grid_constant__ CUtensorMap k_map,
                         const __grid_constant__ CUtensorMap v_map, MqParams mp) {
  const AttnParams& p = mp.a;
  constexpr int D = kED;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* qx = smem + kEStages * kEStageBytes;
  float* m_sh = reinterpret_cast<float*>(qx + kEQxBytes);   // [2][128] the sets' references
  float* l_sh = m_sh + 2 * kERows;                           // [2][128] the sets' row sums
  float* rowc_st = l_sh + 2 * kERows;                        // [128] staged row constants of the next unit
  float* scale_sh = rowc_st + kERows;                        // [stage][4 c, 4 a, 4 1/v, 4 unused]
  int* lens_sh = reinterpret_cast<int*>(scale_sh + kEStages * 16);
  uint16_t* order_sh = reinterpret_cast<uint16_t*>(lens_sh + kEMaxBatch);
  uint64_t* bars = reinterpret_cast<uint64_t*>(order_sh + kEMaxBatch);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kEBars);
  int* cta_err = reinterpret_cast<int*>(tmem_slot + 1);
  int* bad_sh = cta_err + 1;   // [2] by round parity: a page id of the unit was out of range
  int* stop_sh = bad_sh + 2;   // [2] by round parity: a wait has timed out, the softmax warps leave together

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.group, T = mp.n_q;
  const int rows_total = T * G;
  const int n_rb = (rows_total + kERows - 1) / kERows;
  const int n_units = p.batch * p.geom.num_kv_heads * n_rb;
  const bool half_rows = rows_total <= kERows / 2;
  // once any CTA of this launch has reported a timed-out wait, the rest do not start
  if (p.status != nullptr && *reinterpret_cast<volatile int32_t*>(p.status) == PDA_DEV_TIMEOUT) return;

  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kEStages;
  const uint32_t bar_s3 = empty0 + 8 * kEStages, bar_p = bar_s3 + 24, bar_pv = bar_p + 16, bar_buf = bar_pv + 16;
  const uint32_t bar_q = bar_buf + 24, bar_qfull = bar_q + 8, bar_qfree = bar_qfull + 8;
  if (tid == 0) {
    for (int s = 0; s < kEStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);  // released by the PV MMAs' commit
    }
    for (int k = 0; k < kEBufs; ++k) {
      mbar_init(bar_s3 + 8 * k, 1);   // S ready in buffer k
      mbar_init(bar_buf + 8 * k, 1);  // buffer k free again: its P . V has completed
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(bar_p + 8 * k, 4);    // one arrival per warp of the softmax set that owns the iteration
      mbar_init(bar_pv + 8 * k, 1);
    }
    mbar_init(bar_q, kESoftmaxWarps);      // the unit's Q is in tensor memory
    mbar_init(bar_qfull, 1);               // the stager has written a unit's Q parts to shared memory
    mbar_init(bar_qfree, kESoftmaxWarps);  // ... and the softmax warps have taken them out
    *cta_err = 0;
    bad_sh[0] = bad_sh[1] = 0;
    stop_sh[0] = stop_sh[1] = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == kEMmaWarp) {  // tensor memory; this warp also releases it
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(kETmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // lengths, and the order of the sequences by length (longest first, ties by index): order_sh[rank] = j
  for (int j = tid; j < p.batch; j += kEThreads) lens_sh[j] = max(p.seq_lens[j], 0);
  __syncthreads();
  {
    // (one key per sequence, (length << 10) | (1023 - index): distinct and larger for the sequence that
    // comes first; a rank is the number of larger keys, counted four keys to a load. The keys lie in the
    // ring, which no copy has been sent to yet. Lengths from 2^21 on rank as equal.)
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem);
    const int n_keys = (p.batch + 3) & ~3;
    for (int j = tid; j < n_keys; j += kEThreads)
      keys[j] = j < p.batch ? (static_cast<uint32_t>(min(lens_sh[j], (1 << 21) - 1)) << 10) | static_cast<uint32_t>(1023 - j) : 0u;
    __syncthreads();
    for (int j = tid; j < p.batch; j += kEThreads) {
      const uint32_t kj = keys[j];
      int rank = 0;
      for (int i = 0; i < n_keys; i += 4) {
        const uint4 k4 = *reinterpret_cast<const uint4*>(keys + i);
        rank += (k4.x > kj) + (k4.y > kj) + (k4.z > kj) + (k4.w > kj);
      }
      order_sh[rank] = static_cast<uint16_t>(j);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + kETmemO, tmem_q = tmem_base + kETmemQ;
  const int n_cta = gridDim.x, cta = blockIdx.x;

  // The CTA's round-th unit, the same for every warp: positions in the sorted order are dealt in
  // serpentine rounds. false: no more units.
  auto unit_at = [&](int round, EUnit& u) -> bool {
    const int pos = round * n_cta + ((round & 1) ? n_cta - 1 - cta : cta);
    if (pos >= n_units) return false;
    const int per_seq = p.geom.num_kv_heads * n_rb;
    u.b = order_sh[pos / per_seq];
    u.g = (pos % per_seq) / n_rb;
    u.rb = pos % n_rb;
    u.L = lens_sh[u.b];
    u.err = static_cast<int64_t>(u.L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ? PDA_DEV_BAD_SEQ_LEN : 0;
    u.n_pages = u.err ? 0 : (u.L + kPageSize - 1) / kPageSize;
    u.n_iters = (u.n_pages + kEPagesPerIter - 1) / kEPagesPerIter;
    return true;
  };
  auto dead = [&]() { return *reinterpret_cast<volatile int*>(cta_err) == PDA_DEV_TIMEOUT; };

  // ---- stager: the NEXT unit's Q rows, scaled, split into e4m3 high and low parts, into shared memory
  auto stager_role = [&]() {
    // Row r of the unit -> (query token r / G, head r % G). The row times a power of two that brings its
    // largest magnitude into [128, 256), written as hi + lo, both e4m3 (exact for every element within 2^-9 of
    // the largest: a bf16 has 8 significant bits, each part 4); the power goes into the row's score constant.
    const int n_rows = half_rows ? kERows / 2 : kERows;
    EUnit u;
    for (int round = 0; unit_at(round, u); ++round) {
      if (dead()) break;
      if (round > 0 && !__all_sync(0xffffffffu, mbar_wait_bounded(bar_qfree, (round - 1) & 1))) {
        if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
        break;
      }
      for (int t = lane; t < n_rows; t += 32) {
        const int r = u.rb * kERows + t;
        const bool valid = r < rows_total;
        const int64_t qrow = (static_cast<int64_t>(u.b) * T + r / G) * p.num_q_heads + u.g * G + (r % G);
        const uint4* src = reinterpret_cast<const uint4*>(p.q + qrow * D);
        uint32_t amax = 0u;  // bf16 magnitudes order like their bit patterns
#pragma unroll 4
        for (int ch = 0; ch < D / 8; ++ch) {
          const uint4 v = valid ? __ldg(src + ch) : make_uint4(0u, 0u, 0u, 0u);
          const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) amax = max(amax, max((w4[e] << 16) & 0x7fff0000u, w4[e] & 0x7fff0000u));
        }
        const int ex = static_cast<int>(amax >> 23);                      // biased exponent of the largest magnitude
        const int up = (ex == 0 || ex == 255) ? 0 : min(max(134 - ex, -100), 100);  // it times 2^up is in [128, 256)
        const float mul = __uint_as_float(static_cast<uint32_t>(127 + up) << 23);
        rowc_st[t] = p.scale * 1.4426950408889634f * __uint_as_float(static_cast<uint32_t>(127 - up) << 23);
        uint2* dst_hi = reinterpret_cast<uint2*>(qx + t * kEQPitch);
        uint2* dst_lo = reinterpret_cast<uint2*>(qx + t * kEQPitch + 128);
#pragma unroll 2
        for (int ch = 0; ch < D / 8; ++ch) {  // (the second pass over the row comes from L1 / L2)
          const uint4 v = valid ? __ldg(src + ch) : make_uint4(0u, 0u, 0u, 0u);
          const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
          uint32_t h2[4], l2[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float x0 = __uint_as_float(w4[e] << 16) * mul, x1 = __uint_as_float(w4[e] & 0xffff0000u) * mul;
            h2[e] = f32x2_to_e4m3x2(x0, x1);
            uint32_t back16 = e4m3x2_to_f16x2(h2[e]);  // what the tensor core will read for the high parts
            const float2 back = __half22float2(*reinterpret_cast<__half2*>(&back16));
            l2[e] = f32x2_to_e4m3x2(x0 - back.x, x1 - back.y);
          }
          dst_hi[ch] = make_uint2(h2[0] | (h2[1] << 16), h2[2] | (h2[3] << 16));
          dst_lo[ch] = make_uint2(l2[0] | (l2[1] << 16), l2[2] | (l2[3] << 16));
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive_tc(bar_qfull);
    }
  };

  // ---- TMA producer: runs through all units of the CTA, held back only by the ring
  auto producer_role = [&]() {
    const uint32_t leader = elect_one();
    const uint64_t pol = l2_policy_evict_first();  // a sequence's own tiles are read once; a shared prefix stays
                                                   // in the L2 all the same (measured)
    EUnit u;
    uint32_t gi = 0;  // iterations so far, over all units
    bool bad = false, alive = true;
    for (int round = 0; alive && unit_at(round, u); ++round) {
      if (dead()) break;
      const int32_t* table = p.block_table + static_cast<int64_t>(u.b) * p.block_table_stride;
      const int g = u.g;
      int pg = 0;
      // per page: the score factor (K scale), log2 of the V scale and its reciprocal. The scales are positive
      // by construction; the clamps keep an all-zero or negative entry from producing inf or NaN.
      // (lanes past the last page keep finite values: a masked score times 0 would be NaN)
      float sc_c = 1.f, sc_a = 0.f, sc_i = 1.f;
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        const uint32_t s = gi % kEStages;
        if ((it & 7) == 0) {  // page ids of the next 8 iterations (32 pages), one per lane
          pg = 0;
          if (it * kEPagesPerIter + lane < u.n_pages) {
            const int v = table[it * kEPagesPerIter + lane];
            pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
            const float ks = fabsf(p.k_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g]);
            const float vs = fabsf(p.v_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g]);
            const float vc = fminf(fmaxf(vs, 8.6736174e-19f), 1.1529215e18f);  // 2^-60 .. 2^60
            sc_c = fminf(fmaxf(ks, 1e-30f), 1e30f);
            sc_a = __log2f(vc);
            sc_i = 1.f / vc;
          }
        }
        bool ok = true;
        if (gi >= kEStages) ok = mbar_wait_bounded(empty0 + 8 * s, ((gi / kEStages) - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); alive = false; break; }
        const int n_here = min(kEPagesPerIter, u.n_pages - it * kEPagesPerIter);
        const uint32_t stage = ring + s * kEStageBytes, bar = full0 + 8 * s;
        // this stage's page constants, written by the lanes that hold its pages (seen through the full barrier)
        if ((lane >> 2) == (it & 7)) {
          scale_sh[s * 16 + (lane & 3)] = sc_c;
          scale_sh[s * 16 + 4 + (lane & 3)] = sc_a;
          scale_sh[s * 16 + 8 + (lane & 3)] = sc_i;
          scale_sh[s * 16 + 12 + (lane & 3)] = (pg < 0 && (lane & 3) < n_here) ? 1.f : 0.f;  // a bad page id here
        }
        __syncwarp();
        mbar_expect_tx_if(leader, bar, n_here * 2 * kETileBytes);
        auto load_page = [&](int j) {  // an e4m3 row is one 128-byte line: K and V tiles are copied whole
          const int page_raw = __shfl_sync(0xffffffffu, pg, (it & 7) * kEPagesPerIter + j);
          bad |= page_raw < 0;
          const int page = max(page_raw, 0);
          tma_load_5d_hint_if(leader, stage + j * kETileBytes, &k_map, bar, 0, g, page, pol);
          tma_load_5d_hint_if(leader, stage + kEKBytes + j * kETileBytes, &v_map, bar, 0, g, page, pol);
        };
        if (n_here == kEPagesPerIter) {
#pragma unroll
          for (int j = 0; j < kEPagesPerIter; ++j) load_page(j);
        } else {
          for (int j = 0; j < n_here; ++j) load_page(j);
        }
      }
    }
    if (bad && lane == 0) atomicMax(cta_err, PDA_DEV_BAD_PAGE);
  };

  // ---- S issue: S(gi) = Q . K^T as soon as its operands allow
  auto s_issue_role = [&]() {
    constexpr uint32_t idesc_s = tc_idesc(kEPagesPerIter * kPageSize, false, kFmtE4m3, kFmtE4m3);
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    EUnit u;
    uint32_t gi = 0;
    bool ok = true;
    for (int round = 0; ok && unit_at(round, u); ++round) {
      if (dead()) break;
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar_q, round & 1));  // this unit's Q is in tensor memory
      if (!ok) break;
      tc_fence_after();
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        const uint32_t buf = gi % kEBufs, s = gi % kEStages;
        // S(gi) overwrites the buffer of S(gi-3) and P(gi-3): P(gi-3) . V has completed
        // (the stage first: it has landed long ago as a rule, while the buffer is what S waits for)
        ok = mbar_wait_bounded(full0 + 8 * s, (gi / kEStages) & 1);  // the block has landed
        if (ok && gi >= kEBufs) ok = mbar_wait_bounded(bar_buf + 8 * buf, ((gi / kEBufs) - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t stage = ring + s * kEStageBytes;
        const int n_here = min(kEPagesPerIter, u.n_pages - it * kEPagesPerIter);
        const int tail = u.L - (it * kEPagesPerIter + n_here - 1) * kPageSize;  // valid rows of the last page here
        // P is 0 past the sequence end, but V must be finite there: clear those rows of the last page, and
        // (an MMA step spans two pages) the missing second page of the last step
        const bool odd = n_here & 1;
        if (tail < kPageSize || odd) {
          const uint32_t vt = stage + kEKBytes + (n_here - 1) * kETileBytes;
          const int first = max(min(tail, kPageSize), 0) * 128, end = (odd ? 2 : 1) * kETileBytes;
          for (int i = first + lane * 16; i < end; i += 32 * 16)
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + i), "r"(0));
          fence_proxy_async();
          __syncwarp();
        }
        tc_fence_after();
        const uint32_t d = u_tmem + 64 * buf;
        // S[:, 0..64) = Q . K^T over the 64 stacked token rows: contraction over d in 4 steps of 32, once with
        // the high and once with the low parts of Q (descriptor start addresses in 16-byte units: +2 per step)
        // (rows of pages that were not loaded hold stale data: those columns are masked later)
        const uint64_t kd0 = tc_desc(stage, 16, 1024);
#pragma unroll
        for (int part = 0; part < 2; ++part)
#pragma unroll
          for (int ks = 0; ks < D / 32; ++ks)
            tc_mma_ts_if<true>(leader, d, u_tmem + kETmemQ + 32 * part + 8 * ks, kd0 + static_cast<uint64_t>(ks * 2),
                               idesc_s, (part | ks) ? 1u : 0u);
        tc_commit_if(leader, bar_s3 + 8 * buf);
      }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };

  // ---- PV issue: O[set] += P . V
  auto pv_issue_role = [&]() {
    constexpr uint32_t idesc_pv = tc_idesc(D, true, kFmtE4m3, kFmtE4m3);
    constexpr uint32_t idesc_pv_lo = tc_idesc(D, true, kFmtE5m2, kFmtE4m3);  // the low parts of P are e5m2
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    EUnit u;
    uint32_t gi = 0;
    bool ok = true;
    for (int round = 0; ok && unit_at(round, u); ++round) {
      if (dead()) break;
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        const uint32_t set = gi & 1, buf = gi % kEBufs, s = gi % kEStages;
        ok = mbar_wait_bounded(bar_p + 8 * set, (gi >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t stage = ring + s * kEStageBytes;
        const int n_here = min(kEPagesPerIter, u.n_pages - it * kEPagesPerIter);
        const uint32_t pa0 = u_tmem + 64 * buf;
        // V read MN-major: an e4m3 line holds all 128 columns of d; SBO: next 8 tokens
        const uint64_t vd0 = tc_desc(stage + kEKBytes, kPageSize * 128, 1024);
        // O[set] += P[:, 32j .. 32j+32) . V : one K = 32 step per two pages (their tiles are contiguous), once
        // with each of the three parts of P (high, middle: e4m3; low: e5m2). The set's first iteration of a
        // unit (it 0 or 1) starts its accumulator anew.
        auto pv_pair = [&](int j) {
#pragma unroll
          for (int part = 0; part < 3; ++part)
            tc_mma_ts_if<true>(leader, u_tmem + kETmemO + D * set, pa0 + 16 * part + 8 * j,
                               vd0 + static_cast<uint64_t>(j * (2 * kETileBytes / 16)), part == 2 ? idesc_pv_lo : idesc_pv,
                               (it > 1 || j > 0 || part > 0) ? 1u : 0u);
        };
        pv_pair(0);
        if (n_here > 2) pv_pair(1);
        tc_commit_if(leader, empty0 + 8 * s);       // the stage may be refilled once these MMAs have read it
        tc_commit_if(leader, bar_pv + 8 * set);     // O updated
        tc_commit_if(leader, bar_buf + 8 * buf);    // the S / P buffer is free again
      }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  };

  // ---- softmax: TMEM lane t <-> query row t; set x takes the iterations gi with gi % 2 == x, as an online
  // softmax of its own with its own accumulator. kNp = pages of an iteration a thread works on: 4 (its row
  // sees all 64 tokens) or 2 (half rows: lanes below 64 take tokens 0..31, lanes from 64 tokens 32..63 of
  // the same query rows).
  auto softmax_role = [&](auto pages_tag) {
    constexpr int kNp = decltype(pages_tag)::value;
    constexpr bool kHalf = kNp == 2;
    constexpr int kNc = kNp * kPageSize;  // columns (tokens) per thread and iteration
    const int set = warp >> 2, t = tid & (kERows - 1);
    const int half = kHalf ? (t >> 6) : 0;  // warp-uniform
    const int qr = kHalf ? (t & (kERows / 2 - 1)) : t;  // row within the unit's block
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;  // this warp's TMEM lanes
    const uint32_t my_p = bar_p + 8 * set, my_pv = bar_pv + 8 * set;
    EUnit u;
    uint32_t g0 = 0;  // iterations of the units before this one
    bool alive = true;
    auto fail = [&]() { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); alive = false; };
    // (A warp that gives up on a wait still goes through the unit's named barriers -- the other softmax
    // warps are waiting there without a limit -- and all eight leave together on the stop flag.)
    for (int round = 0; unit_at(round, u); ++round) {
      // ---- this unit's Q: from the stage to tensor memory (this warp: 64 of the row's 128 elements, by set)
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_qfull, round & 1))) fail();
      float rowc = 0.f;
      if (alive) {
        uint32_t qh[16], ql[16];
        const uint4* sh = reinterpret_cast<const uint4*>(qx + qr * kEQPitch + 64 * set);
        const uint4* sl = reinterpret_cast<const uint4*>(qx + qr * kEQPitch + 128 + 64 * set);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 a = sh[i], b4 = sl[i];
          qh[4 * i] = a.x; qh[4 * i + 1] = a.y; qh[4 * i + 2] = a.z; qh[4 * i + 3] = a.w;
          ql[4 * i] = b4.x; ql[4 * i + 1] = b4.y; ql[4 * i + 2] = b4.z; ql[4 * i + 3] = b4.w;
        }
        rowc = rowc_st[qr];
        const uint32_t my_q = tmem_q + lane_base;
        tmem_st16(my_q + 16 * set, qh);
        tmem_st16(my_q + 32 + 16 * set, ql);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_tc(bar_q);      // the S issue warp may start on this unit
          mbar_arrive_tc(bar_qfree);  // the stager may write the next unit's rows
        }
      }
      const int r = u.rb * kERows + qr;
      const int i_tok = r / G;
      const int lim = mp.causal ? min(u.L, u.L - T + i_tok + 1) : u.L;
      const int n_iters = u.n_iters;
      const int it0 = (set ^ static_cast<int>(g0 & 1));  // this set's first iteration of the unit
      float m_ref = -INFINITY;   // reference the accumulated O is scaled by
      float l_set = 0.f, m_l = -INFINITY;  // this thread's share of the row sum and the reference it is scaled by
      bool bad_unit = false;
      for (int it = it0; alive && it < n_iters; it += 2) {
        const uint32_t gi = g0 + it;
        const uint32_t buf = gi % kEBufs, sc_stage = gi % kEStages;
        bool ok = mbar_spin_bounded(bar_s3 + 8 * buf, (gi / kEBufs) & 1);  // S(gi)
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        uint32_t sv[kNc];
        const uint32_t sp_buf = tmem_s + 64 * buf + lane_base;
        if constexpr (kHalf) {
          tmem_ld32(sp_buf + 32 * half, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        } else {
          tmem_ld32(sp_buf, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32(sp_buf + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        }
        tmem_wait_ld();
        const int tok0 = it * kEPagesPerIter * kPageSize + kNc * half;  // first token of this thread's columns
        const int n_vis = lim - tok0;  // visible ones among them (may be <= 0)
        if (__any_sync(0xffffffffu, n_vis < kNc)) {  // boundary tiles only
#pragma unroll
          for (int j = 0; j < kNc; ++j) sv[j] = (j < n_vis) ? sv[j] : 0xff800000u;  // -inf
        }
        // per page q of the thread's columns: x = s cq + aq with cq = K scale x row constant and aq = log2 of the
        // V scale: the softmax runs on the scores plus log2(V scale), so P carries the V scale into P . V (V is
        // multiplied as raw e4m3), and the page's sum of P divided by the V scale (iq) is its share of l.
        // (the constants were written by the producer before the tiles' full barrier completed, which the
        // S issue warp observed before the MMAs whose commit this warp has waited for)
        float cq[kNp], aq[kNp], iq[kNp];
        {
          const float4 bf = *reinterpret_cast<const float4*>(scale_sh + sc_stage * 16 + 12);
          bad_unit |= (bf.x + bf.y + bf.z + bf.w) != 0.f;
          const float* sc = scale_sh + sc_stage * 16 + kNp * half;
#pragma unroll
          for (int q = 0; q < kNp; ++q) {
            cq[q] = fmaxf(sc[q] * rowc, 1e-37f);  // (kept above zero: a masked score, -inf, times 0 would be NaN)
            aq[q] = sc[4 + q];
            iq[q] = sc[8 + q];
          }
        }
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
        // set kERefBelowMax under the maximum (the three 8-bit parts of a weight are exact from 2^-6 up)
        float m_new = m_ref;
        if (mx > m_ref + kERescaleThreshold || m_ref == -INFINITY) m_new = mx - kERefBelowMax;
        const bool need = m_new != m_ref && m_ref != -INFINITY;
        if (it > 1 && __any_sync(0xffffffffu, need)) {
          // O may only be touched once this set's last PV into it, PV(gi-2), has completed; PV(gi) is not
          // issued before this warp arrives on bar_p below
          ok = mbar_spin_bounded(my_pv, ((gi >> 1) - 1) & 1);
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
        if (gi >= 2) {
          // (P goes over its own S; this wait keeps the set's view of the barrier one phase behind at most,
          // which the parity waits on it rely on)
          ok = mbar_spin_bounded(my_pv, ((gi >> 1) - 1) & 1);
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

      // ---- finalise the unit: this set's last PV, then the merge of the accumulators that hold parts of a
      // row: the two sets' (and, with half rows, those of lanes r and r + 64)
      bool ok = alive;
      if (alive && n_iters > it0) {
        const uint32_t gl = g0 + (n_iters - 1 - ((n_iters - 1 - it0) & 1));  // this set's last iteration
        ok = __all_sync(0xffffffffu, mbar_wait_bounded(my_pv, (gl >> 1) & 1));
        if (!ok) fail();
        tc_fence_after();
      }
      if (m_l != m_ref) l_set *= ex2(m_l - m_ref);
      m_sh[set * kERows + t] = m_ref;
      l_sh[set * kERows + t] = l_set;
      if (bad_unit && lane == 0) bad_sh[round & 1] = 1;
      if ((!alive || dead()) && lane == 0) stop_sh[round & 1] = 1;
      // every softmax warp reaches this point with its error view settled; all P . V of the unit have completed
      asm volatile("bar.sync 2, %0;" ::"n"(kESoftmaxWarps * 32) : "memory");
      const bool timed_out = stop_sh[round & 1] != 0;  // the same for all eight warps
      if (tid == 0) {  // (the next unit's flags: nobody touches them before that unit's finalisation)
        bad_sh[(round + 1) & 1] = 0;
        stop_sh[(round + 1) & 1] = 0;
      }
      const int dev_err = max(u.err, max(bad_sh[round & 1] ? PDA_DEV_BAD_PAGE : 0, timed_out ? PDA_DEV_TIMEOUT : 0));
      if (dev_err && tid == 0) report(p.status, dev_err);
      const bool valid_row = r < rows_total;
      const bool have = n_iters > 0 && !timed_out;  // CTA-uniform
      const bool has0 = n_iters > static_cast<int>(g0 & 1), has1 = n_iters > static_cast<int>((g0 & 1) ^ 1);  // set 0 / 1 took part
      float l = 0.f, w0 = 0.f, w1 = 0.f;  // weights of this lane's two accumulators (one per set)
      float m_row = -INFINITY;
      if (have) {
        const float m0 = m_sh[t], m1 = m_sh[kERows + t];
        float M = fmaxf(m0, m1);
        const int tp = t ^ (kERows / 2);  // half rows: the lane that holds the row's other half
        if constexpr (kHalf) M = fmaxf(M, fmaxf(m_sh[tp], m_sh[kERows + tp]));
        auto wgt = [&](float m) { return m == -INFINITY ? 0.f : ex2(m - M); };
        w0 = wgt(m0);
        w1 = wgt(m1);
        l = w0 * l_sh[t] + w1 * l_sh[kERows + t];
        if constexpr (kHalf) l += wgt(m_sh[tp]) * l_sh[tp] + wgt(m_sh[kERows + tp]) * l_sh[kERows + tp];
        m_row = M;
      }
      const bool live = !dev_err && have && l > 0.f;
      const float inv = live ? 1.f / l : 0.f;
      // set x handles columns [D/2 x, D/2 (x + 1)) of the row, 32 at a time: this lane's accumulators, weighted
      uint32_t ov[D / 64][32];
#pragma unroll
      for (int cc = 0; cc < D / 64; ++cc) {
        const int cb = (D / 64) * set + cc;
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[cc][j] = 0u;
        if (have && has0) {
          tmem_ld32(tmem_o + lane_base + 32 * cb, ov[cc]);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) ov[cc][j] = __float_as_uint(__uint_as_float(ov[cc][j]) * w0);
        }
        if (have && has1) {
          uint32_t o1[32];
          tmem_ld32(tmem_o + D + lane_base + 32 * cb, o1);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j)
            ov[cc][j] = __float_as_uint(fmaf(__uint_as_float(o1[j]), w1, __uint_as_float(ov[cc][j])));
        }
      }
      tc_fence_before();
      if constexpr (kHalf) {
        // lanes from 64 hand their part to the lane that stores the row, 32 columns per set at a time, through
        // the second half of the Q staging area ([set][column][row]: a warp's lanes write consecutive words)
        float* xch = reinterpret_cast<float*>(qx + kEQxBytes / 2);  // (16 KB of that area)
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {
          if (half == 1) {
#pragma unroll
            for (int j = 0; j < 32; ++j) xch[(set * 32 + j) * (kERows / 2) + qr] = __uint_as_float(ov[cc][j]);
          }
          asm volatile("bar.sync 2, %0;" ::"n"(kESoftmaxWarps * 32) : "memory");
          if (half == 0) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              ov[cc][j] = __float_as_uint(__uint_as_float(ov[cc][j]) + xch[(set * 32 + j) * (kERows / 2) + qr]);
          }
          // (also the unit's closing barrier: every read of the accumulators, of m_sh / l_sh and of the
          // exchange area lies before it, every write of the next unit after it)
          asm volatile("bar.sync 2, %0;" ::"n"(kESoftmaxWarps * 32) : "memory");
        }
      } else {
        asm volatile("bar.sync 2, %0;" ::"n"(kESoftmaxWarps * 32) : "memory");  // the unit's closing barrier
      }
      if constexpr (kHalf) {
        // The rows leave through shared memory (the exchange area is free again): a thread holds 64 columns
        // of one row, so stored directly a warp's instruction would touch 32 rows; from shared memory every
        // 16 lanes write one row's 256 bytes.
        uint8_t* ostage = qx + kEQxBytes / 2;
        if (half == 0) {
          uint4* dst = reinterpret_cast<uint4*>(ostage + qr * kEQPitch + 128 * set);
#pragma unroll
          for (int cc = 0; cc < D / 64; ++cc)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e)
                w[e] = pack2<false>(__uint_as_float(ov[cc][8 * j + 2 * e]) * inv,
                                    __uint_as_float(ov[cc][8 * j + 2 * e + 1]) * inv);
              dst[4 * cc + j] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kESoftmaxWarps * 32) : "memory");
#pragma unroll
        for (int k = 0; k < (kERows / 2) * 16 / (kESoftmaxWarps * 32); ++k) {
          const int chunk = tid + k * kESoftmaxWarps * 32;  // 16-byte piece of the 64 x 256 bytes
          const int row = chunk >> 4, piece = chunk & 15;
          const int rr = u.rb * kERows + row;
          if (rr < rows_total) {
            const int64_t orow = (static_cast<int64_t>(u.b) * T + rr / G) * p.num_q_heads + u.g * G + (rr % G);
            *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(p.out + orow * D) + 16 * piece) =
                *reinterpret_cast<const uint4*>(ostage + row * kEQPitch + 16 * piece);
          }
        }
      } else if (valid_row) {
        const int64_t qrow = (static_cast<int64_t>(u.b) * T + i_tok) * p.num_q_heads + u.g * G + (r % G);
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {
          const int cb = (D / 64) * set + cc;
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
      (void)m_row;
      g0 += static_cast<uint32_t>(n_iters);
      if (timed_out) break;
    }
  };

  // by warpgroup, each first taking or giving up registers
  if (warp < kESoftmaxWarps) {
    reg_alloc_inc<kERegsSoftmax>();
    if (half_rows) softmax_role(std::integral_constant<int, 2>{});
    else softmax_role(std::integral_constant<int, 4>{});
  } else {
    reg_alloc_dec<kERegsControl>();
    if (warp == kEProducerWarp) producer_role();
    else if (warp == kEMmaWarp) s_issue_role();
    else if (warp == kEPvWarp) pv_issue_role();
    else stager_role();
  }

  // ---- teardown: everyone is done with tensor memory before it is released
  tc_fence_before();
  __syncthreads();
  if (warp == kEMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kETmemCols) : "memory");
  }
}

}  // namespace

bool attention_mq_tc8p_supports(const MqParams& mp) {
  const AttnParams& p = mp.a;
  if (p.geom.dtype != PDA_FP8_E4M3 || p.geom.head_dim != kED || p.k_scale == nullptr || p.v_scale == nullptr) return false;
  if (p.chunk_tokens > 0 || mp.kv_len_fixed != 0 || p.first_token != 0 || p.window > 0) return false;
  if (p.group < 1 || mp.n_q < 1 || p.geom.num_pages < 1 || p.batch < 1 || p.batch > kEMaxBatch) return false;
  if (!(p.scale > 0.f) || !(p.scale < INFINITY)) return false;  // the row maximum is taken before scaling
  return true;
}

cudaError_t launch_attention_mq_tc8p(const MqParams& mp, cudaStream_t stream) {
  const AttnParams& p = mp.a;
  alignas(64) CUtensorMap k_map, v_map;
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, 1) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, 1))
    return cudaErrorNotSupported;
  cudaError_t e = cudaFuncSetAttribute(attention_mq_tc8p_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kESmemBytes);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int rows_total = mp.n_q * p.group;
  const int64_t n_units = static_cast<int64_t>(p.batch) * p.geom.num_kv_heads * ((rows_total + kERows - 1) / kERows);
  // with a unit or less per SM there is nothing to carry from one unit to the next, and the one-unit kernel
  // starts faster (32 units: 34.7 against 42.1 us; 144 units: 39.6 against 43.5; 192 units: 65.1 against 63.9)
  if (n_units <= sms && attention_mq_tc_supports(mp)) return launch_attention_mq_tc(mp, stream);
  const unsigned grid = static_cast<unsigned>(n_units < sms ? n_units : sms);  // one CTA per SM
  attention_mq_tc8p_kernel<<<grid, kEThreads, kESmemBytes, stream>>>(k_map, v_map, mp);
  return cudaGetLastError();
}

}  // namespace pda
