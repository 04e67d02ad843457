// Multi-query paged attention on tcgen05 + TMEM, persistent CTAs: the tiles, warp roles and barrier
// chains of attention_mq_tc.cu (bf16 KV, head_dim 128, unsplit), but one CTA per SM walks through many
// (sequence, kv head, row block) units instead of one CTA per unit. A unit's start and drain cost the
// one-CTA-per-unit kernel about 6 us (set-up, ranking, a trip to memory for Q, another for the first
// tiles, the last P.V, the output), a fifth to a third of a unit at the lengths of a decode batch. Here
//   - barriers, tensor memory and the order of the sequences are set up once per CTA;
//   - the TMA producer runs on into the next unit's tiles while the current unit drains (12 stages ahead);
//   - the next unit's Q rows are fetched during the current unit's last iterations and stored to tensor
//     memory as soon as its last S has completed, so the S of the next unit is computed while the last
//     P.V and the output of the current one are under way.
// Units are ordered by the length of their sequence (longest first; all of a sequence's units next to one
// another). Most are dealt to the CTAs in serpentine order, so that every CTA works on a mix of long and
// short units; the shortest ones are claimed from a counter in device memory, so that a CTA whose share
// was long draws fewer of them. The counter is one of a small pool the library owns; the CTA that leaves
// last puts it back to zero.
// Iterations are numbered through all units of a CTA (gi); ring stages, S/P buffers, softmax sets and
// barrier phases follow gi as they follow the iteration index in the one-unit kernel.
#include <atomic>
#include <mutex>

#include "common.cuh"
#include "tma_ptx.cuh"
#include "tcgen05_ptx.cuh"

namespace pda {

namespace {

constexpr int kPRows = kUmmaRows;
constexpr int kPPagesPerIter = 4;      // 64 tokens per iteration
constexpr int kPD = 128;
constexpr int kPLines = kPD / 64;
constexpr int kPTileBytes = kPageSize * kPD * 2;             // 4096
constexpr int kPKBytes = kPPagesPerIter * kPTileBytes;       // K of 4 pages as [lines][64 tokens][128 B]
constexpr int kPStageBytes = 2 * kPKBytes;                   // K block, then 4 V page tiles: 32 KB
constexpr int kPStages = 6;
constexpr int kPOnesBytes = 2048;                            // bf16 ones: B operand of the row-sum MMA
constexpr int kPMBytes = 2 * kPRows * 4;                     // running row maxima handed between the softmax sets
constexpr int kPMaxBatch = 1024;                             // lengths and order of the sequences in shared memory
constexpr int kPSortBatch = 352;                             // sorted up to one sequence per thread
constexpr int kPLensBytes = kPMaxBatch * 4, kPOrderBytes = kPMaxBatch * 2;
constexpr int kPSmemBytes = kPStages * kPStageBytes + kPOnesBytes + kPMBytes + kPLensBytes + kPOrderBytes + 128 + 512 + 1024;
constexpr int kPSoftmaxWarps = 8, kPProducerWarp = 8, kPMmaWarp = 9, kPPvWarp = 10;
constexpr int kPThreads = 352;
constexpr uint32_t kPTmemCols = 512;
constexpr uint32_t kPTmemO = 128, kPTmemQ = 256, kPTmemP = 320, kPTmemL = 384;
constexpr float kPRescaleThreshold = 8.f;

// Units are claimed from a counter in device memory (longest sequences first) by the producer warp, which
// is the first to need them, and handed to the other warps through a small ring in shared memory: entry k
// holds the position of the CTA's k-th unit in the sorted order, or -1 when there are no more. Only units
// with iterations go through the ring (the producer writes the zero rows of an empty sequence itself), so
// the producer is never more than kPStages + 2 entries ahead of the slowest reader.
constexpr int kPClaimRing = 16;
constexpr int kPClaimedRounds = 3;
__device__ __forceinline__ void publish_unit(volatile int* ring_sh, int k, int pos) {  // one thread
  ring_sh[2 * (k % kPClaimRing) + 1] = pos;
  __threadfence_block();
  ring_sh[2 * (k % kPClaimRing)] = k + 1;  // tag: entry k is valid
}
__device__ __forceinline__ int unit_entry(volatile int* ring_sh, int k, int lane) {  // a whole warp; -2: timed out
  int pos = -2;
  if (lane == 0) {
    for (uint32_t i = 0; i < (1u << 23); ++i) {  // (64 ns naps: gives up after about a second)
      if (ring_sh[2 * (k % kPClaimRing)] == k + 1) {
        __threadfence_block();
        pos = ring_sh[2 * (k % kPClaimRing) + 1];
        break;
      }
      __nanosleep(64);
    }
  }
  return __shfl_sync(0xffffffffu, pos, 0);
}

__global__ void __launch_bounds__(kPThreads, 1)
attention_mq_tcp_kernel(const __grid_constant__ CUtensorMap k_map,
                        const __grid_constant__ CUtensorMap v_map, MqParams mp, unsigned int* claim) {
  const AttnParams& p = mp.a;
  constexpr int D = kPD;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ones_smem = smem + kPStages * kPStageBytes;
  float* m_sh = reinterpret_cast<float*>(ones_smem + kPOnesBytes);              // [2][128]
  int* lens_sh = reinterpret_cast<int*>(m_sh + 2 * kPRows);                      // [batch]
  uint16_t* order_sh = reinterpret_cast<uint16_t*>(lens_sh + kPMaxBatch);        // [batch]: longest first
  int* ring_sh = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(order_sh) + kPOrderBytes);  // [kPClaimRing][tag, position]
  // full[], empty[], s[2], p[2], pv[2], sfree[2], m[2][4], qready, ofree
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring_sh + 2 * kPClaimRing);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kPStages + 18);
  int* cta_err = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = p.group, T = mp.n_q;
  const int rows_total = T * G;
  const int n_rb = (rows_total + kPRows - 1) / kPRows;
  const int per_seq = p.geom.num_kv_heads * n_rb;   // units of a sequence
  const int n_units = p.batch * per_seq;
  const int cta = blockIdx.x, n_ctas = gridDim.x;
  // The claim counter is zero between launches: the CTA that leaves last puts it back.
  auto leave = [&]() {
    if (threadIdx.x == 0 && atomicAdd(&claim[1], 1u) == gridDim.x - 1) {
      claim[0] = 0u;
      claim[1] = 0u;
      __threadfence();
    }
  };
  // once any CTA of this launch has reported a timed-out wait, the rest do not start
  if (p.status != nullptr && *reinterpret_cast<volatile int32_t*>(p.status) == PDA_DEV_TIMEOUT) {
    leave();
    return;
  }

  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kPStages;
  const uint32_t bar_s = empty0 + 8 * kPStages, bar_p = bar_s + 16, bar_pv = bar_p + 16;  // two of each
  const uint32_t bar_sfree = bar_pv + 16, bar_m = bar_sfree + 16, bar_qready = bar_m + 64, bar_ofree = bar_qready + 8;
  for (int i = tid; i < kPOnesBytes / 4; i += kPThreads)
    reinterpret_cast<uint32_t*>(ones_smem)[i] = 0x3F803F80u;  // 1.0 as bf16 pairs
  fence_proxy_async();  // read by the tensor core through the async proxy
  if (tid == 0) {
    for (int s = 0; s < kPStages; ++s) {
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
    mbar_init(bar_qready, 4);               // a unit's Q is in tensor memory (stored by one softmax set)
    mbar_init(bar_ofree, 4);                // a unit's O and l have been read (by the set that owns its last iteration)
    for (int i = 0; i < 2 * kPClaimRing; ++i) ring_sh[i] = 0;
    *cta_err = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  if (warp == kPMmaWarp) {  // tensor memory; this warp also releases it
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(kPTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // lengths, and the order of the sequences: longest first (ties by index) up to kPSortBatch sequences
  for (int j = tid; j < p.batch; j += kPThreads) lens_sh[j] = max(p.seq_lens[j], 0);
  __syncthreads();
  if (p.batch <= kPSortBatch) {
    // (one key per sequence, (length << 9) | (511 - index): distinct and larger for the sequence that comes
    // first; a rank is the number of larger keys, counted four keys to a load. The keys lie in the ring,
    // which no copy has been sent to yet. Lengths from 2^22 on rank as equal.)
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem);
    const int n_keys = (p.batch + 3) & ~3;
    for (int j = tid; j < n_keys; j += kPThreads)
      keys[j] = j < p.batch ? (static_cast<uint32_t>(min(lens_sh[j], (1 << 22) - 1)) << 9) | static_cast<uint32_t>(511 - j) : 0u;
    __syncthreads();
    if (tid < p.batch) {
      const uint32_t kj = keys[tid];
      int rank = 0;
      for (int i = 0; i < n_keys; i += 4) {
        const uint4 k4 = *reinterpret_cast<const uint4*>(keys + i);
        rank += (k4.x > kj) + (k4.y > kj) + (k4.z > kj) + (k4.w > kj);
      }
      order_sh[rank] = static_cast<uint16_t>(tid);
    }
  } else {
    for (int j = tid; j < p.batch; j += kPThreads) order_sh[j] = static_cast<uint16_t>(j);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + kPTmemO;  // S buffer k at tmem_s + 64 k
  const uint32_t tmem_q = tmem_base + kPTmemQ, tmem_p = tmem_base + kPTmemP;  // P buffer k at tmem_p + 32 k

  // A unit: sequence b, kv head g, row block rb; its pages and iterations (0 if its length does not fit the
  // block table, which is reported).
  struct Unit { int b, g, rb, L, n_pages, n_iters; bool bad; };
  auto unit_at = [&](int pos) {
    Unit u;
    const int sp = pos / per_seq, rem = pos % per_seq;
    u.b = order_sh[sp];
    u.g = rem / n_rb;
    u.rb = rem % n_rb;
    u.L = lens_sh[u.b];
    u.bad = static_cast<int64_t>(u.L) > static_cast<int64_t>(p.block_table_stride) * kPageSize;
    u.n_pages = u.bad ? 0 : (u.L + kPageSize - 1) / kPageSize;
    u.n_iters = (u.n_pages + kPPagesPerIter - 1) / kPPagesPerIter;
    return u;
  };

  if (warp == kPProducerWarp) {
    // ================= TMA producer: runs through the units' tiles, up to kPStages iterations ahead ====
    const uint32_t leader = elect_one();
    const uint64_t pol = l2_policy_evict_first();  // the tiles are read once: first out of the L2
    bool bad = false, dead = false;
    uint32_t gi = 0;
    // (a quarter of the rounds, at most kPClaimedRounds: with only three or four units a CTA the deal is as
    // even as claiming, and claiming would make every CTA work on units of like length at any one time)
    const int dealt_rounds = n_units / n_ctas - min(kPClaimedRounds, n_units / n_ctas / 4);
    int n_dealt = 0;
    for (int k = 0; !dead;) {
      // The first rounds are dealt in serpentine order over the sorted units (every CTA works on a mix of long
      // and short units, which keeps the HBM busy while some CTAs are between units); the shortest units, the
      // last kPClaimedRounds rounds' worth, are claimed from the counter and even out the CTAs' ends.
      int pos = 0;
      if (n_dealt < dealt_rounds) {
        pos = n_dealt * n_ctas + ((n_dealt & 1) ? n_ctas - 1 - cta : cta);
        ++n_dealt;
      } else {
        if (lane == 0) pos = dealt_rounds * n_ctas + static_cast<int>(atomicAdd(&claim[0], 1u));
        pos = __shfl_sync(0xffffffffu, pos, 0);
      }
      if (pos >= n_units) {
        if (lane == 0) publish_unit(ring_sh, k, -1);
        break;
      }
      const Unit u = unit_at(pos);
      if (u.n_iters == 0) {  // an empty (or misdescribed) sequence: its output rows are zero, written here
        if (u.bad && lane == 0) report(p.status, PDA_DEV_BAD_SEQ_LEN);
        for (int rr = lane; rr < kPRows; rr += 32) {
          const int r = u.rb * kPRows + rr;
          if (r < rows_total) {
            uint4* dst = reinterpret_cast<uint4*>(
                p.out + ((static_cast<int64_t>(u.b) * T + r / G) * p.num_q_heads + u.g * G + (r % G)) * D);
#pragma unroll
            for (int j = 0; j < D / 8; ++j) dst[j] = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        continue;
      }
      if (lane == 0) publish_unit(ring_sh, k, pos);
      ++k;
      const int32_t* table = p.block_table + static_cast<int64_t>(u.b) * p.block_table_stride;
      // The producer reaches a unit some iterations before the softmax warps fetch its Q rows: it sends them
      // towards L2 now (a load from DRAM takes about 3000 clocks while the other SMs stream).
      if (gi > 0) {
        for (int rr = lane; rr < kPRows; rr += 32) {
          const int r = u.rb * kPRows + rr;
          if (r < rows_total) {
            const __nv_bfloat16* row = p.q + ((static_cast<int64_t>(u.b) * T + r / G) * p.num_q_heads + u.g * G + (r % G)) * D;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(row + D / 2));
          }
        }
      }
      int pg = 0;
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        const uint32_t s = gi % kPStages;
        if ((it & 7) == 0) {  // page ids of the next 8 iterations (32 pages), one per lane
          pg = 0;
          if (it * kPPagesPerIter + lane < u.n_pages) {
            const int v = table[it * kPPagesPerIter + lane];
            pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
          }
        }
        bool ok = true;
        if (gi >= kPStages) ok = mbar_wait_bounded(empty0 + 8 * s, ((gi / kPStages) - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); dead = true; break; }
        const int n_here = min(kPPagesPerIter, u.n_pages - it * kPPagesPerIter);
        const uint32_t stage = ring + s * kPStageBytes, bar = full0 + 8 * s;
        mbar_expect_tx_if(leader, bar, n_here * 2 * kPTileBytes);
        // K: one copy per 128-byte line so that page j's 16 rows follow page j-1's in each line block
        auto load_page = [&](int j) {
          const int page_raw = __shfl_sync(0xffffffffu, pg, (it & 7) * kPPagesPerIter + j);
          bad |= page_raw < 0;
          const int page = max(page_raw, 0);
#pragma unroll
          for (int ln = 0; ln < kPLines; ++ln)
            tma_load_5d_hint_if(leader, stage + ln * (kPKBytes / kPLines) + j * (kPageSize * 128), &k_map, bar, ln, u.g, page, pol);
          tma_load_5d_hint_if(leader, stage + kPKBytes + j * kPTileBytes, &v_map, bar, 0, u.g, page, pol);
        };
        if (n_here == kPPagesPerIter) {
#pragma unroll
          for (int j = 0; j < kPPagesPerIter; ++j) load_page(j);
        } else {
          for (int j = 0; j < n_here; ++j) load_page(j);
        }
      }
    }
    if (bad && lane == 0) atomicMax(cta_err, PDA_DEV_BAD_PAGE);
  } else if (warp == kPMmaWarp) {
    // ================= S issue: S(gi) = Q . K^T as soon as its operands allow =================
    constexpr uint32_t idesc_s = tc_idesc(kPPagesPerIter * kPageSize, false, kFmtBf16, kFmtBf16);
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    bool ok = true;
    uint32_t gi = 0;
    for (int k = 0; ok; ++k) {
      const int pos = unit_entry(ring_sh, k, lane);
      if (pos < 0) { ok = pos == -1; break; }
      const Unit u = unit_at(pos);
      // this unit's Q is in tensor memory (the softmax warps store it once the previous unit's last S is done)
      ok = mbar_wait_bounded(bar_qready, k & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        const uint32_t stage_i = gi % kPStages;
        // S(gi) overwrites the buffer of S(gi-2): the softmax warps have loaded that into registers
        if (gi >= 2) ok = mbar_wait_bounded(bar_sfree + 8 * (gi & 1), ((gi - 2) >> 1) & 1);
        if (ok) ok = mbar_wait_bounded(full0 + 8 * stage_i, (gi / kPStages) & 1);  // the block has landed
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t stage = ring + stage_i * kPStageBytes;
        const int n_here = min(kPPagesPerIter, u.n_pages - it * kPPagesPerIter);
        const int tail = u.L - (it * kPPagesPerIter + n_here - 1) * kPageSize;  // valid rows of the last page here
        if (tail < kPageSize) {  // P is 0 past the sequence end, but V must be finite there
          const uint32_t vt = stage + kPKBytes + (n_here - 1) * kPTileBytes;
          constexpr int kChunksPerRow = D / 8;  // 16-byte chunks of a row
          for (int i = lane; i < (kPageSize - tail) * kChunksPerRow; i += 32) {
            const int r = tail + i / kChunksPerRow, ch = i % kChunksPerRow;
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_off(r, ch)), "r"(0));
          }
          fence_proxy_async();
          __syncwarp();
        }
        tc_fence_after();
        const uint32_t d = u_tmem + 64 * (gi & 1);
        // S[:, 0..64) = Q . K^T over the 64 stacked token rows, contraction over d in steps of 16
        // (rows of pages that were not loaded hold stale data: those columns are masked later)
        const uint64_t kd0 = tc_desc(stage, 16, 1024);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t bd = kd0 + static_cast<uint64_t>((ks >> 2) * (kPKBytes / kPLines / 16) + (ks & 3) * 2);
          tc_mma_ts_if<false>(leader, d, u_tmem + kPTmemQ + 8 * ks, bd, idesc_s, ks > 0 ? 1u : 0u);
        }
        tc_commit_if(leader, bar_s + 8 * (gi & 1));
      }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  } else if (warp == kPPvWarp) {
    // ================= PV issue: O += P . V and l += P . 1 =================
    constexpr uint32_t idesc_pv = tc_idesc(D, true, kFmtBf16, kFmtBf16);
    constexpr uint32_t idesc_l = tc_idesc(16, false, kFmtBf16, kFmtBf16);
    const uint64_t ones_desc = tc_desc(smem_u32(ones_smem), 16, 1024);
    const uint32_t leader = elect_one();
    const uint32_t u_tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
    bool ok = true;
    uint32_t gi = 0;
    for (int k = 0; ok; ++k) {
      const int pos = unit_entry(ring_sh, k, lane);
      if (pos < 0) { ok = pos == -1; break; }
      const Unit u = unit_at(pos);
      for (int it = 0; it < u.n_iters; ++it, ++gi) {
        ok = mbar_wait_bounded(bar_p + 8 * (gi & 1), (gi >> 1) & 1);
        // the unit's first PV overwrites O and l: every softmax warp has read the previous unit's
        if (ok && it == 0 && k > 0) ok = mbar_wait_bounded(bar_ofree, (k - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t stage_i = gi % kPStages;
        const uint32_t stage = ring + stage_i * kPStageBytes;
        const int n_here = min(kPPagesPerIter, u.n_pages - it * kPPagesPerIter);
        const uint32_t pa0 = u_tmem + kPTmemP + 32 * (gi & 1);
        // V read MN-major. LBO: next 64 columns of d, SBO: next 8 tokens
        const uint64_t vd0 = tc_desc(stage + kPKBytes, kPageSize * 128, 1024);
        // O += P[:, 16j .. 16j+16) . V_j : one K = 16 step per page
        // and l += P[:, 16j .. 16j+16) . 1 : the row sums of exactly the P that multiplies V
        auto pv_page = [&](int j) {
          const uint32_t acc = (it > 0 || j > 0) ? 1u : 0u;
          tc_mma_ts_if<false>(leader, u_tmem + kPTmemO, pa0 + 8 * j, vd0 + static_cast<uint64_t>(j * (kPTileBytes / 16)), idesc_pv, acc);
          tc_mma_ts_if<false>(leader, u_tmem + kPTmemL, pa0 + 8 * j, ones_desc, idesc_l, acc);
        };
        if (n_here == kPPagesPerIter) {
#pragma unroll
          for (int j = 0; j < kPPagesPerIter; ++j) pv_page(j);
        } else {
          for (int j = 0; j < n_here; ++j) pv_page(j);
        }
        tc_commit_if(leader, empty0 + 8 * stage_i);     // the stage may be refilled once these MMAs have read it
        tc_commit_if(leader, bar_pv + 8 * (gi & 1));    // O and l updated, P buffer free again
      }
    }
    if (!ok && lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  } else {
    // ================= softmax: TMEM lane t <-> query row t; set x takes the iterations gi with gi % 2 == x
    const int set = warp >> 2, t = tid & (kPRows - 1);
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;  // this warp's TMEM lanes
    const float scale_log2 = p.scale * 1.4426950408889634f;
    const uint32_t my_s = bar_s + 8 * set, my_p = bar_p + 8 * set, my_pv = bar_pv + 8 * set;
    const uint32_t my_sfree = bar_sfree + 8 * set;
    // the running maximum passes between the two warps that own the same 32 rows (same scheduler)
    const uint32_t my_m = bar_m + 8 * (4 * set + (warp & 3)), other_m = bar_m + 8 * (4 * (set ^ 1) + (warp & 3));
    bool alive = true;
    auto fail = [&]() { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); alive = false; };
    // Q of a unit: row r -> (query token r / G, head r % G) goes to TMEM lane r as the A operand of
    // S = Q . K^T. One softmax set loads and stores the whole rows: at the end of a unit the set that does
    // not own the last iteration, which is done one iteration earlier than the other (a load takes about
    // 2500 clocks while the other SMs stream, from L2 as well as from DRAM).
    auto load_q = [&](int pos_q, uint32_t last_s) {
      const Unit u = unit_at(pos_q);
      const int r = u.rb * kPRows + t;
      const bool valid = r < rows_total;
      const int64_t qrow = (static_cast<int64_t>(u.b) * T + r / G) * p.num_q_heads + u.g * G + (r % G);
      const uint4* src = reinterpret_cast<const uint4*>(p.q + qrow * D);
      uint32_t qreg[D / 2];
#pragma unroll
      for (int ch = 0; ch < D / 8; ++ch) {
        const uint4 v = valid ? src[ch] : make_uint4(0u, 0u, 0u, 0u);
        qreg[4 * ch] = v.x; qreg[4 * ch + 1] = v.y; qreg[4 * ch + 2] = v.z; qreg[4 * ch + 3] = v.w;
      }
      bool ok = true;
      if (last_s != 0xffffffffu) {  // the previous unit's last S has completed: its Q is no longer read
        ok = mbar_spin_bounded(bar_s + 8 * (last_s & 1), (last_s >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
      }
      if (ok) {
#pragma unroll
        for (int h = 0; h < D / 64; ++h) {
          uint32_t part[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) part[j] = qreg[32 * h + j];
          tmem_st32(tmem_q + lane_base + 32 * h, part);
        }
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_tc(bar_qready);
      }
      return ok;
    };
    int pos = unit_entry(ring_sh, 0, lane);  // the CTA's first unit
    if (pos == -2) fail();
    if (pos >= 0 && set == 0) load_q(pos, 0xffffffffu);
    uint32_t gi0 = 0;  // first iteration of the unit
    for (int k = 0; alive && pos >= 0; ++k) {
      const Unit u = unit_at(pos);
      const int r = u.rb * kPRows + t;
      const bool valid_row = r < rows_total;
      const int i_tok = r / G;
      const int64_t qrow = (static_cast<int64_t>(u.b) * T + i_tok) * p.num_q_heads + u.g * G + (r % G);
      const int L = u.L;
      const int lim = mp.causal ? min(L, L - T + i_tok + 1) : L;
      float m_ref = -INFINITY;   // reference max the accumulated O and l (both in tensor memory) are scaled by
      for (int it = ((gi0 & 1u) == static_cast<uint32_t>(set)) ? 0 : 1; it < u.n_iters; it += 2) {
        const uint32_t gi = gi0 + it;
        const uint32_t ph = (gi >> 1) & 1;  // phase of this set's barriers at this iteration
        bool ok = mbar_spin_bounded(my_s, ph);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        uint32_t sv[2][32];
        tmem_ld32(tmem_s + 64 * set + lane_base, sv[0]);
        tmem_ld32(tmem_s + 64 * set + lane_base + 32, sv[1]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_tc(my_sfree);  // S(gi) is in registers: S(gi+2) may overwrite its buffer
        const int tok0 = it * kPPagesPerIter * kPageSize;
        const int n_vis = lim - tok0;  // visible columns of this row in this iteration (may be <= 0)
        if (__any_sync(0xffffffffu, n_vis < kPPagesPerIter * kPageSize)) {  // boundary tiles only
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
        // the reference after the unit's previous iteration comes from the other set
        if (it > 0) {
          ok = mbar_spin_bounded(other_m, ((gi - 1) >> 1) & 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { fail(); break; }
          m_ref = m_sh[((gi - 1) & 1) * kPRows + t];
        }
        // lazy rescaling: keep the old reference unless the max grew past the threshold
        float m_new = m_ref;
        if (mx > m_ref + kPRescaleThreshold || m_ref == -INFINITY) m_new = fmaxf(m_ref, mx);
        const bool need = m_new != m_ref && m_ref != -INFINITY;
        m_sh[(gi & 1) * kPRows + t] = m_new;
        __syncwarp();
        if (lane == 0) mbar_arrive_tc(my_m);  // (release: the other set reads m_sh after its wait)
        if (it > 0 && __any_sync(0xffffffffu, need)) {
          // O and l may only be touched once PV(gi-1) has completed; PV(gi) is not issued before this
          // warp arrives on bar_p below, and the other set rescales only after PV(gi)
          // (a parity wait tells neighbouring phases apart only: first this set's own PV(gi-2), after which
          // the other set's barrier cannot be more than one phase behind)
          if (gi >= 2) ok = mbar_spin_bounded(my_pv, ph ^ 1);
          if (ok) ok = mbar_spin_bounded(bar_pv + 8 * (set ^ 1), ((gi - 1) >> 1) & 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { fail(); break; }
          tc_fence_after();
          const float alpha = need ? ex2(m_ref - m_new) : 1.f;
#pragma unroll
          for (int cb = 0; cb < D / 32 + 1; ++cb) {  // O, then the block of columns that holds l
            uint32_t ov[32];
            tmem_ld32(tmem_o + lane_base + (cb < D / 32 ? 32 * cb : kPTmemL - kPTmemO), ov);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
            tmem_st32(tmem_o + lane_base + (cb < D / 32 ? 32 * cb : kPTmemL - kPTmemO), ov);
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
          pw[j] = pack2<false>(ex2(x0), ex2(x1));
        }
        if (gi >= 2) {  // PV(gi-2) has finished reading the P buffer this iteration writes
          ok = mbar_spin_bounded(my_pv, ph ^ 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) { fail(); break; }
        }
        tmem_st32(tmem_p + 32 * set + lane_base, pw);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_tc(my_p);
      }
      if (!alive) break;

      // ---- the unit's end, shared out between the sets. The set that does not own the last iteration is
      // done one iteration earlier: it loads the next unit's Q and goes on to that unit, whose first
      // iteration is its own. The set that owns the last iteration waits for the last PV and writes the
      // whole rows of the output while the other set is already at work on the next unit.
      const uint32_t glast = gi0 + u.n_iters - 1;
      bool ok = true;
      int pos_next;  // the CTA's next unit (claimed by the producer some iterations ago), or -1
      if ((glast & 1) != static_cast<uint32_t>(set)) {
        pos_next = unit_entry(ring_sh, k + 1, lane);
        if (pos_next == -2 || (pos_next >= 0 && !load_q(pos_next, glast))) { fail(); break; }
        // (the owner's last running maximum is not needed, but its barrier phase is consumed here: a parity
        // wait only tells neighbouring phases apart)
        ok = mbar_spin_bounded(bar_m + 8 * (4 * (glast & 1) + (warp & 3)), (glast >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
      } else {
        ok = mbar_spin_bounded(my_pv, (glast >> 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { fail(); break; }
        tc_fence_after();
        uint32_t l_bits;
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(l_bits) : "r"(tmem_base + kPTmemL + lane_base));
        tmem_wait_ld();
        const float l = __uint_as_float(l_bits);
        const float inv = l > 0.f ? 1.f / l : 0.f;
        uint32_t w[D / 2];  // the row as bf16 pairs
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
          uint32_t ov[32];
          tmem_ld32(tmem_o + lane_base + 32 * cb, ov);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            w[16 * cb + j] = pack2<false>(__uint_as_float(ov[2 * j]) * inv, __uint_as_float(ov[2 * j + 1]) * inv);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_tc(bar_ofree);  // O and l are in registers: the next unit's first PV may overwrite them
        if (valid_row) {
          uint4* dst = reinterpret_cast<uint4*>(p.out + qrow * D);
#pragma unroll
          for (int j = 0; j < D / 8; ++j) dst[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        }
        pos_next = unit_entry(ring_sh, k + 1, lane);
        if (pos_next == -2) { fail(); break; }
      }
      gi0 += u.n_iters;
      pos = pos_next;
    }
  }

  // ---- teardown: everyone is done with tensor memory before it is released
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *cta_err) report(p.status, *cta_err);
  if (warp == kPMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kPTmemCols) : "memory");
  }
  leave();
}

}  // namespace

bool attention_mq_tcp_supports(const MqParams& mp) {
  const AttnParams& p = mp.a;
  if (p.geom.dtype != PDA_BF16 || p.geom.head_dim != kPD) return false;
  if (p.chunk_tokens > 0 || mp.kv_len_fixed != 0 || p.first_token != 0 || p.window > 0) return false;
  if (p.group < 1 || mp.n_q < 1 || p.geom.num_pages < 1 || p.batch < 1 || p.batch > kPMaxBatch) return false;
  if (!(p.scale > 0.f) || !(p.scale < INFINITY)) return false;  // the row maximum is taken before scaling
  return true;
}

namespace {
// Claim counters: [next unit, CTAs that have left] each, zero between launches. Launches take the slots in
// turn, so that launches running side by side on different streams do not share one (up to kClaimSlots of
// them); a captured launch keeps the slot it was captured with.
constexpr int kClaimSlots = 64, kClaimDevices = 64;
__device__ unsigned int g_claim[kClaimSlots][4];
std::atomic<unsigned> g_claim_next{0};
std::mutex g_claim_mu;
unsigned int* g_claim_base[kClaimDevices] = {};
cudaError_t claim_counter(int dev, unsigned int** out) {
  if (dev < 0 || dev >= kClaimDevices) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(g_claim_mu);
    if (g_claim_base[dev] == nullptr) {
      void* ptr = nullptr;
      if (cudaError_t e = cudaGetSymbolAddress(&ptr, g_claim)) return e;
      g_claim_base[dev] = static_cast<unsigned int*>(ptr);
    }
  }
  *out = g_claim_base[dev] + 4 * (g_claim_next.fetch_add(1) % kClaimSlots);
  return cudaSuccess;
}
}  // namespace

cudaError_t launch_attention_mq_tcp(const MqParams& mp, cudaStream_t stream) {
  const AttnParams& p = mp.a;
  alignas(64) CUtensorMap k_map, v_map;
  // K is copied one 128-byte line of its rows at a time (so that the pages of an iteration stack), V as whole tiles
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, 2, /*box_lines=*/1) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, 2))
    return cudaErrorNotSupported;
  cudaError_t e = cudaFuncSetAttribute(attention_mq_tcp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemBytes);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int rows_total = mp.n_q * p.group;
  const int n_rb = (rows_total + kPRows - 1) / kPRows;
  const int64_t n_units = static_cast<int64_t>(p.batch) * p.geom.num_kv_heads * n_rb;
  // with a unit or less per SM there is nothing to carry from one unit to the next
  if (n_units <= sms && attention_mq_tc_supports(mp)) return launch_attention_mq_tc(mp, stream);
  const unsigned grid = static_cast<unsigned>(n_units < sms ? n_units : sms);
  unsigned int* claim = nullptr;
  if ((e = claim_counter(dev, &claim)) != cudaSuccess) return e;
  attention_mq_tcp_kernel<<<grid, kPThreads, kPSmemBytes, stream>>>(k_map, v_map, mp, claim);
  return cudaGetLastError();
}

}  // namespace pda
