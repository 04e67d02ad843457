// Paged decode attention for sm_100a: TMA page gather + tensor-core GQA tiles.
//
// Work item = (sequence b, kv head g, chunk c) = one CTA of kWarps warps. Every
// warp is a self-contained flash-decoding worker: it owns a ring of kStages
// shared-memory stages, each one (page, kv head) K tile plus V tile, filled by
// 5-D tiled TMA copies (128-byte swizzle) that complete on the warp's own
// mbarriers, so the steady state has no CTA-wide synchronisation. Warp w takes
// the chunk's pages w, w+kWarps, ...; the warps' (m, l, O) states are merged
// through shared memory once at the end.
//
// Per 16-token page tile, with the G <= 8 query heads of the group as the N
// dimension of mma.sync.m16n8k16 (tokens are M, so a page is exactly one MMA
// row block and nothing is padded along the streamed dimension):
//   S^T[16 x 8]  = K_tile[16 x D] . Q_g^T[D x 8]          (D/16 MMAs)
//   online softmax over tokens (max by shuffles across the 8 row groups)
//   O^T[D x 8]  += V_tile^T[D x 16] . P^T[16 x 8]          (D/16 MMAs)
// K fragments come from ldmatrix, V^T fragments from ldmatrix.trans, P^T is
// turned from accumulator layout into B-operand layout by movmatrix. e4m3 tiles
// are converted to f16 in registers (cvt.rn.f16x2.e4m3x2, exact); their
// per-(page, head) scales multiply the scores (K) and the probabilities (V).
//
// The tile math lives in decode_tile.cuh. The same kernel is the fused decode step
// (paged_decode_step): the warp that owns the sequence's last page patches the new token's
// K/V rows into the landed tile and stores them to the cache (append); split units publish
// their partial and the unit's last-arriving chunk (atomic count in the caller's workspace)
// merges them all; unsplit launches serve the longest sequences first. A token range
// (first_token, window) restricts the attended tokens; pages wholly outside it are not read.
//
// Every wait on an mbarrier is bounded; on expiry the CTA reports
// PDA_DEV_TIMEOUT, waits (bounded) for its copies in flight and zero-fills its
// output. TMA copies never use multicast.
#include <atomic>

#include "common.cuh"
#include "decode_tile.cuh"
#include "tma_ptx.cuh"

namespace pda {

namespace {

// ---- kernel ------------------------------------------------------------------------------

constexpr int kMaxLptBatch = 256;  // above this the O(batch^2 / threads) ranking costs more than it saves

template <int D, bool kFp8, int kStages, int kWarps>
struct Cfg {
  static constexpr int kElem = kFp8 ? 1 : 2;
  static constexpr int kRowBytes = D * kElem;            // one token row
  static constexpr int kTileBytes = kPageSize * kRowBytes;
  static constexpr int kStageBytes = 2 * kTileBytes;     // K tile then V tile
  static constexpr int kWarpRing = kStages * kStageBytes;
  static constexpr int kKSteps = D / 16;                 // MMAs of each product per tile
  static constexpr int kOStride = D + 4;                 // fp32 row pitch of the merge buffer
  static constexpr int kMergeBytes = (8 * kOStride + 16) * 4;
  static constexpr int kSmemBytes = kWarps * kWarpRing + kWarps * kStages * 8 + 16 + 1024;
  static_assert(kRowBytes % 128 == 0, "rows must be whole 128-byte swizzle lines");
  static_assert(kMergeBytes <= kWarpRing, "merge buffer reuses the warp's ring");
};

template <int D, bool kFp8, int kStages, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
attention_tma_kernel(const __grid_constant__ CUtensorMap k_map,
                     const __grid_constant__ CUtensorMap v_map, StepParams sp, int longest_first) {
  using C = Cfg<D, kFp8, kStages, kWarps>;
  const AttnParams& p = sp.a;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kWarps * C::kWarpRing);
  int* cta_err = reinterpret_cast<int*>(bars + kWarps * kStages);  // [0] error code, [1] "last chunk of the unit"

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tq = lane & 3;
  const int c = blockIdx.x, g = blockIdx.y;
  int b = blockIdx.z;
  int L_ranked = -1;  // the unit's length when the ranking below has it at hand (saves a trip to memory)
  if (longest_first) {  // (the host: unsplit, 2 .. kMaxLptBatch sequences, few units per resident CTA)
    // unsplit units differ in length by the spread of seq_lens: serve the longest first. The CTA
    // with blockIdx.z = r takes the sequence at place r of an order by decreasing length, so long units
    // start early and short ones fill the tail. (Split units are bounded by chunk_tokens already. With more
    // than about four units per resident CTA the order costs more than it gives: units of like length then
    // run side by side and start side by side, and the HBM idles while they do. Measured on random lengths
    // of 32..2048, bf16, one CTA per unit: 160 sequences 6.05 TB/s in this order, 6.33 as they come; 192:
    // 6.24 and 6.53; 256: 6.50 and 6.62; at 128 sequences, 3.5 units per resident CTA, the order gives 6 %.)
    // Every CTA does this on its way to its first tile, so it has to be cheap: counting, for every sequence,
    // the sequences that come before it cost a 256-sequence launch 22 of 122 us (and 8-10 % from 160
    // sequences up even four keys to a load). Instead: 64 buckets by length (longer first; the bucket
    // width is the largest length / 64 rounded up to a power of two), by index inside a bucket. A warp
    // handles 32 consecutive sequences at a time and finds a sequence's place among those of its bucket
    // with a match; the counts per (32 sequences, bucket) are summed up by one warp. Every CTA computes the
    // same order. 128 threads, up to 256 sequences: two per thread.
    static_assert(kWarps == 4 && kMaxLptBatch == 256, "two sequences per thread, chunks of 32 by warp");
    int* hist = reinterpret_cast<int*>(smem);   // [8 chunks][64 buckets]: sequences of the bucket in the chunk,
                                                // then: in the chunks before it
    int* offset = hist + 8 * 64;                // [64] sequences in the buckets above
    int* wmax = offset + 64;                    // [4]
    int l_mine[2];
    int lmax = 0;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int j = tid + 128 * k;
      l_mine[k] = j < p.batch ? max(p.seq_lens[j], 0) : 0;
      lmax = max(lmax, l_mine[k]);
    }
    for (int i = tid; i < 8 * 64; i += 128) hist[i] = 0;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) lmax = max(lmax, __shfl_xor_sync(0xffffffffu, lmax, off));
    if (lane == 0) wmax[warp] = lmax;
    __syncthreads();
    lmax = max(max(wmax[0], wmax[1]), max(wmax[2], wmax[3]));
    const int shift = max(32 - __clz(lmax) - 6, 0);  // lmax >> shift < 64
    int bkt[2], ord[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int j = tid + 128 * k;
      bkt[k] = j < p.batch ? (l_mine[k] >> shift) : 64 + lane;  // (no sequence: a bucket of its own, not counted)
      const unsigned same = __match_any_sync(0xffffffffu, bkt[k]);
      ord[k] = __popc(same & ((1u << lane) - 1u));
      if (ord[k] == 0 && j < p.batch) hist[(warp + 4 * k) * 64 + bkt[k]] = __popc(same);
    }
    __syncthreads();
    if (warp == 0) {
      int tot[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {  // buckets lane and lane + 32: counts -> counts in the chunks before
        int run = 0;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          const int x = hist[ch * 64 + lane + 32 * h];
          hist[ch * 64 + lane + 32 * h] = run;
          run += x;
        }
        tot[h] = run;
      }
      int s_lo = tot[0], s_hi = tot[1];  // -> sums over the buckets from this one up, within each half
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int y_lo = __shfl_down_sync(0xffffffffu, s_lo, off), y_hi = __shfl_down_sync(0xffffffffu, s_hi, off);
        if (lane + off < 32) { s_lo += y_lo; s_hi += y_hi; }
      }
      const int all_hi = __shfl_sync(0xffffffffu, s_hi, 0);
      offset[lane + 32] = s_hi - tot[1];
      offset[lane] = s_lo - tot[0] + all_hi;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int j = tid + 128 * k;
      if (j < p.batch && offset[bkt[k]] + hist[(warp + 4 * k) * 64 + bkt[k]] + ord[k] == static_cast<int>(blockIdx.z)) {
        cta_err[2] = j;
        cta_err[3] = l_mine[k];
      }
    }
    __syncthreads();
    b = cta_err[2];
    L_ranked = cta_err[3];
    __syncthreads();  // lens aliases the ring: done with it before any copy lands
  }
  const int G = p.group;
  const bool split = p.chunk_tokens > 0;
  const int64_t row0 = static_cast<int64_t>(b) * p.num_q_heads + static_cast<int64_t>(g) * G;

  // fused step: this launch also writes `out` (merging split-KV partials through the
  // workspace's per-unit chunk counters) and applies the append
  const bool fuse = sp.fuse_reduce != 0;
  const int L = L_ranked >= 0 ? L_ranked : max(p.seq_lens[b], 0);
  int t0 = p.first_token, t1 = L;
  if (split) {
    t0 = p.first_token + c * p.chunk_tokens;
    if (t0 >= L) {
      if (fuse && c == 0)  // empty sequence: its output rows are zero
        for (int i = tid; i < G * D; i += kWarps * 32) p.out[row0 * D + i] = __float2bfloat16_rn(0.f);
      return;
    }
    t1 = min(t0 + p.chunk_tokens, L);
  }
  const int nch = split ? min((L - p.first_token + p.chunk_tokens - 1) / p.chunk_tokens,
                              p.max_chunks - p.chunk_slot0) : 1;
  // first attended token of this unit: the chunk start, raised by the sliding window
  const int lo = (p.window > 0 && L - p.window > t0) ? L - p.window : t0;
  int err = 0;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ||
      (split && static_cast<int64_t>(L - p.first_token) >
                    static_cast<int64_t>(p.max_chunks - p.chunk_slot0) * p.chunk_tokens))
    err = PDA_DEV_BAD_SEQ_LEN;

  if (tid == 0) { cta_err[0] = 0; cta_err[1] = 0; }
  const int page0 = lo / kPageSize;  // first page touched (lo need not be page-aligned)
  const int n_tiles = (err || lo >= t1) ? 0 : (t1 + kPageSize - 1) / kPageSize - page0;
  const int n_mine = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;  // tiles warp, warp+kWarps, ...

  const uint32_t ring = smem_u32(smem + warp * C::kWarpRing);
  const uint32_t bar0 = smem_u32(bars + warp * kStages);
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    fence_mbar_init();
    fence_proxy_async();
  }
  __syncthreads();  // also orders the cta_err reset

  // ---- page ids (and e4m3 scales) for this warp's tiles, 32 ordinals per register block
  const int32_t* table = p.block_table + static_cast<int64_t>(b) * p.block_table_stride;
  bool bad_page = false;  // warp-uniform
  auto load_block = [&](int blk, int& pg, float& ks, float& vs) {
    const int kk = blk * 32 + lane;
    pg = 0; ks = 0.f; vs = 0.f;
    if (kk < n_mine) {
      const int v = table[page0 + warp + kk * kWarps];
      pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;  // -1 marks a bad id; clamped where it is used
      if (kFp8) {
        ks = p.k_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g];
        vs = p.v_scale[static_cast<int64_t>(max(pg, 0)) * p.geom.num_kv_heads + g];
      }
    }
  };
  int pgA, pgB; float ksA, ksB, vsA, vsB;
  load_block(0, pgA, ksA, vsA);
  load_block(1, pgB, ksB, vsB);

  const uint32_t leader = elect_one();
  const uint64_t pol = l2_policy_evict_first();
  auto issue = [&](int s, int page_raw) {  // into stage s; whole warp, converged; the elected lane issues
    const int page = max(page_raw, 0);
    const uint32_t bar = bar0 + 8 * s;
    const uint32_t dst = ring + s * C::kStageBytes;
    mbar_expect_tx_if(leader, bar, C::kStageBytes);
    tma_load_5d_hint_if(leader, dst, &k_map, bar, 0, g, page, pol);
    tma_load_5d_hint_if(leader, dst + C::kTileBytes, &v_map, bar, 0, g, page, pol);
  };

  // prologue: fill the ring
  {
    const int n_pre = min(kStages, n_mine);
    for (int kk = 0; kk < n_pre; ++kk) {
      const int page = __shfl_sync(0xffffffffu, pgA, kk);
      if (page < 0) bad_page = true;
      issue(kk, page);
    }
  }
  const bool append_here = sp.k_new != nullptr && !err && L > 0 && c == nch - 1;
  if (!kFp8 && append_here && n_tiles == 0 && warp == 0) {
    // nothing of this unit is attended (the range starts past the new token): append only
    const int v = table[(L - 1) / kPageSize];
    if (v >= 0 && v < p.geom.num_pages) {
      if (lane < C::kRowBytes / 16) {
        const int64_t src = (static_cast<int64_t>(b) * p.geom.num_kv_heads + g) * D + lane * 8;
        const int64_t dst = v * p.geom.page_stride + g * p.geom.head_stride +
                            ((L - 1) % kPageSize) * p.geom.slot_stride + lane * 8;
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(sp.k_cache_w) + dst) =
            *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.k_new) + src);
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(sp.v_cache_w) + dst) =
            *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.v_new) + src);
      }
    } else {
      bad_page = true;
    }
  }

  // ---- Q^T fragments of this unit's group, resident in registers for the whole unit
  uint32_t qf[C::kKSteps][2];
  load_q_fragments<D, kFp8>(p.q + row0 * D, G, gid, tq, qf);

  const float scale_log2 = p.scale * 1.4426950408889634f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2tq, 2tq+1
  float o[C::kKSteps][4];
#pragma unroll
  for (int i = 0; i < C::kKSteps; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

  bool timed_out = false;
  int kk = 0;
  int s = 0;           // kk % kStages and the parity of kk / kStages, kept by counting (the kernel's
  uint32_t phase = 0;  // instructions are what bounds it on e4m3 caches whose pages are shared)
  int tok0 = (page0 + warp) * kPageSize;
  for (; kk < n_mine; ++kk, tok0 += kWarps * kPageSize) {
    const uint32_t bar = bar0 + 8 * s;
    if (!mbar_wait_bounded(bar, phase)) { timed_out = true; break; }
    const uint32_t kt = ring + s * C::kStageBytes, vt = kt + C::kTileBytes;
    const int n_valid = min(kPageSize, t1 - tok0);  // rows [n_skip, n_valid) of the tile are attended
    const int n_skip = max(lo - tok0, 0);           // > 0 only in the unit's first tile
    float ksc = 1.f, vsc = 1.f;
    if (kFp8) {
      ksc = __shfl_sync(0xffffffffu, ksA, kk & 31);
      vsc = __shfl_sync(0xffffffffu, vsA, kk & 31);
    }

    if (!kFp8 && append_here && warp + kk * kWarps == n_tiles - 1) {
      // fused append: the new token's K/V rows go into the landed tile and into the cache
      const int slot = (L - 1) % kPageSize;
      const int page = __shfl_sync(0xffffffffu, pgA, kk & 31);
      if (lane < C::kRowBytes / 16 && page >= 0) {
        const int64_t src = (static_cast<int64_t>(b) * p.geom.num_kv_heads + g) * D + lane * 8;
        const uint4 kv = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.k_new) + src);
        const uint4 vv = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.v_new) + src);
        const int64_t dst = page * p.geom.page_stride + g * p.geom.head_stride +
                            slot * p.geom.slot_stride + lane * 8;
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(sp.k_cache_w) + dst) = kv;
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(sp.v_cache_w) + dst) = vv;
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(kt + tile_off(slot, lane)),
                     "r"(kv.x), "r"(kv.y), "r"(kv.z), "r"(kv.w));
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(vt + tile_off(slot, lane)),
                     "r"(vv.x), "r"(vv.y), "r"(vv.z), "r"(vv.w));
      }
      __syncwarp();
    }
    decode_tile<D, kFp8>(kt, vt, n_valid, n_skip, scale_log2 * ksc, vsc, qf, m0, m1, l0, l1, o, lane);

    // ---- hand the stage back: every lane has consumed its fragments
    __syncwarp();
    const int kn = kk + kStages;
    if (((kk + 1) & 31) == 0) {  // the consumer moves to the next register block
      pgA = pgB; ksA = ksB; vsA = vsB;
      load_block((kk + 1) / 32 + 1, pgB, ksB, vsB);
    }
    if (kn < n_mine) {
      // kn lies in the consumer's block or the one after it
      const bool in_a = (kn >> 5) == ((kk + 1) >> 5);
      const int page = __shfl_sync(0xffffffffu, in_a ? pgA : pgB, kn & 31);
      if (page < 0) bad_page = true;
      fence_proxy_async();
      issue(s, page);  // (kn % kStages == kk % kStages)
    }
    if (++s == kStages) { s = 0; phase ^= 1u; }
  }

  if (timed_out) {
    // give the copies still in flight a bounded chance to land before the CTA's memory is reused
    for (int j = kk; j < min(kk + kStages, n_mine); ++j)
      mbar_wait_bounded(bar0 + 8 * (j % kStages), (j / kStages) & 1);
    if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT);
  }
  if (bad_page && lane == 0) atomicMax(cta_err, PDA_DEV_BAD_PAGE);

  // ---- publish this warp's state into its own (drained) ring
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  float* mo = reinterpret_cast<float*>(smem + warp * C::kWarpRing);
  float* mm = mo + 8 * C::kOStride;  // m[8] then l[8]
  __syncwarp();
  if (!timed_out) {
    if (gid == 0) {
      mm[2 * tq] = m0; mm[2 * tq + 1] = m1;
      mm[8 + 2 * tq] = l0; mm[8 + 2 * tq + 1] = l1;
    }
    if (2 * tq < G) {
#pragma unroll
      for (int mt = 0; mt < C::kKSteps; ++mt) {
        const int d0 = kFp8 ? 16 * mt + 2 * gid : 16 * mt + gid;
        const int d1 = kFp8 ? d0 + 1 : d0 + 8;
        mo[(2 * tq) * C::kOStride + d0] = o[mt][0];
        mo[(2 * tq + 1) * C::kOStride + d0] = o[mt][1];
        mo[(2 * tq) * C::kOStride + d1] = o[mt][2];
        mo[(2 * tq + 1) * C::kOStride + d1] = o[mt][3];
      }
    }
  }
  __syncthreads();

  // ---- merge the warps' states and write the unit's result
  const int dev_err = max(err, *cta_err);
  if (dev_err && tid == 0) report(p.status, dev_err);
  constexpr float kLn2 = 0.6931471805599453f;
  for (int idx = tid; idx < G * D; idx += kWarps * 32) {
    const int h = idx / D, d = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float* wm = reinterpret_cast<const float*>(smem + w * C::kWarpRing) + 8 * C::kOStride;
      M = fmaxf(M, wm[h]);
    }
    float acc = 0.f, lsum = 0.f;
    if (!dev_err && M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float* wo = reinterpret_cast<const float*>(smem + w * C::kWarpRing);
        const float* wm = wo + 8 * C::kOStride;
        const float mw = wm[h];
        const float wgt = (mw > -INFINITY) ? ex2(mw - M) : 0.f;
        lsum = fmaf(wm[8 + h], wgt, lsum);
        if (wgt != 0.f) acc = fmaf(wo[h * C::kOStride + d], wgt, acc);
      }
    }
    const bool live = !dev_err && lsum > 0.f;
    const float val = live ? acc / lsum : 0.f;
    if (split && !(fuse && nch == 1)) {
      const int64_t pr = (row0 + h) * p.max_chunks + p.chunk_slot0 + c;
      p.part_o[pr * D + d] = val;
      if (d == 0) p.part_lse[pr] = live ? (M + __log2f(lsum)) * kLn2 : -INFINITY;
    } else {
      p.out[(row0 + h) * D + d] = __float2bfloat16_rn(val);
    }
  }

  if (fuse && split && nch > 1) {
    // ---- fused reduce: publish this chunk, count it in; the unit's last chunk merges them all.
    // No CTA waits for another one: whoever arrives last finds every partial already visible.
    int* counter = sp.workspace + 2 + b * p.geom.num_kv_heads + g;
    __threadfence();
    __syncthreads();
    if (tid == 0) cta_err[1] = (atomicAdd(counter, 1) == nch - 1) ? 1 : 0;
    __syncthreads();
    if (cta_err[1]) {
      __threadfence();
      // The merge is the tail of the unit (and, for the last unit, of the launch), so it is spread over
      // the whole CTA with every load independent of the others: a warp per head turns the chunks'
      // log-sum-exps into weights in shared memory (the TMA rings are idle by now), then a thread per
      // (head, 4 columns) accumulates the chunks' partial rows with 16-byte loads.
      float* w_sh = reinterpret_cast<float*>(smem);  // [G][nch] weights, then [G] 1 / sum
      const bool fits = static_cast<int64_t>(G) * (nch + 1) * 4 <= static_cast<int64_t>(kWarps) * C::kWarpRing;
      if (fits) {
        for (int h = warp; h < G; h += kWarps) {
          const float* lse = p.part_lse + (row0 + h) * p.max_chunks + p.chunk_slot0;
          float M = -INFINITY;
          for (int cc = lane; cc < nch; cc += 32) M = fmaxf(M, __ldcg(lse + cc));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
          float W = 0.f;
          for (int cc = lane; cc < nch; cc += 32) {
            const float w = M > -INFINITY ? __expf(__ldcg(lse + cc) - M) : 0.f;
            w_sh[h * nch + cc] = w;
            W += w;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) W += __shfl_xor_sync(0xffffffffu, W, o);
          if (lane == 0) w_sh[G * nch + h] = W > 0.f ? 1.f / W : 0.f;
        }
        __syncthreads();
        constexpr int kVec = D / 4;
        for (int idx = tid; idx < G * kVec; idx += kWarps * 32) {
          const int h = idx / kVec, d4 = idx % kVec;
          const int64_t row = row0 + h;
          const float4* po = reinterpret_cast<const float4*>(p.part_o + (row * p.max_chunks + p.chunk_slot0) * D) + d4;
          const float* wh = w_sh + h * nch;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
          for (int cc = 0; cc < nch; ++cc) {
            const float4 v = __ldcg(po + static_cast<int64_t>(cc) * kVec);
            const float w = wh[cc];
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
          }
          const float inv = w_sh[G * nch + h];
          uint2 packed;
          packed.x = pack2<false>(acc.x * inv, acc.y * inv);
          packed.y = pack2<false>(acc.z * inv, acc.w * inv);
          *reinterpret_cast<uint2*>(p.out + row * D + 4 * d4) = packed;
        }
      } else {
      for (int idx = tid; idx < G * D; idx += kWarps * 32) {
        const int h = idx / D, d = idx % D;
        const int64_t row = row0 + h;
        const float* lse = p.part_lse + row * p.max_chunks + p.chunk_slot0;
        float M = -INFINITY;
        for (int cc = 0; cc < nch; ++cc) M = fmaxf(M, __ldcg(lse + cc));
        float acc = 0.f, W = 0.f;
        if (M > -INFINITY) {
          const float* po = p.part_o + (row * p.max_chunks + p.chunk_slot0) * D + d;
          for (int cc = 0; cc < nch; ++cc) {
            const float w = __expf(__ldcg(lse + cc) - M);
            W += w;
            acc = fmaf(w, __ldcg(po + static_cast<int64_t>(cc) * D), acc);
          }
          acc /= W;
        }
        p.out[row * D + d] = __float2bfloat16_rn(acc);
      }
      }
      if (tid == 0) *counter = 0;  // leave the workspace clean for the next call
    }
  }
}

// ---- host side ---------------------------------------------------------------------------

template <int D, bool kFp8, int kStages, int kWarps>
cudaError_t launch(const StepParams& sp, cudaStream_t stream) {
  using C = Cfg<D, kFp8, kStages, kWarps>;
  const AttnParams& p = sp.a;
  alignas(64) CUtensorMap k_map, v_map;
  const int eb = p.geom.dtype == PDA_BF16 ? 2 : 1;
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb))
    return cudaErrorNotSupported;
  auto kern = attention_tma_kernel<D, kFp8, kStages, kWarps>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const unsigned chunks = p.chunk_tokens > 0 ? static_cast<unsigned>(p.max_chunks - p.chunk_slot0) : 1u;
  dim3 grid(chunks, p.geom.num_kv_heads, p.batch);
  int longest_first = 0;
  if (p.chunk_tokens == 0 && p.batch > 1 && p.batch <= kMaxLptBatch) {
    static std::atomic<int> resident_per_sm{0};  // of this instance of the kernel (the same on every device of a process)
    int per_sm = resident_per_sm.load();
    if (per_sm == 0) {
      if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kWarps * 32, C::kSmemBytes)) != cudaSuccess) return e;
      resident_per_sm.store(per_sm);
    }
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    longest_first = static_cast<int64_t>(p.batch) * p.geom.num_kv_heads <= 4ll * sms * per_sm;
  }
  kern<<<grid, kWarps * 32, C::kSmemBytes, stream>>>(k_map, v_map, sp, longest_first);
  return cudaGetLastError();
}

}  // namespace

namespace {
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no libcuda link).
EncodeFn encode_fn() {
  static EncodeFn fn = [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      sym = nullptr;
    return reinterpret_cast<EncodeFn>(sym);
  }();
  return fn;
}
}  // namespace

bool make_cache_tensor_map(CUtensorMap* map, const void* base, int64_t page_stride,
                           int64_t head_stride, int64_t slot_stride, int num_pages,
                           int num_kv_heads, int head_dim, int eb, int box_lines) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t line_elems = 128 / eb;
  const cuuint64_t lines = static_cast<cuuint64_t>(head_dim) * eb / 128;
  cuuint64_t dims[5] = {line_elems, static_cast<cuuint64_t>(kPageSize), lines,
                        static_cast<cuuint64_t>(num_kv_heads), static_cast<cuuint64_t>(num_pages)};
  cuuint64_t strides[4] = {static_cast<cuuint64_t>(slot_stride) * eb, 128,
                           static_cast<cuuint64_t>(head_stride) * eb,
                           static_cast<cuuint64_t>(page_stride) * eb};
  cuuint32_t box[5] = {static_cast<cuuint32_t>(line_elems), kPageSize,
                       static_cast<cuuint32_t>(box_lines > 0 ? box_lines : lines), 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const CUresult r = enc(map, eb == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 5,
                         const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool attention_tma_supports(const AttnParams& p) {
  if (p.group < 1 || p.group > 8) return false;
  if (p.geom.num_kv_heads > 65535) return false;
  if (p.geom.num_pages < 1) return false;
  if (p.geom.dtype == PDA_BF16) return p.geom.head_dim == 64 || p.geom.head_dim == 128;
  return p.geom.head_dim == 128;
}

cudaError_t launch_step_tma(const StepParams& sp, cudaStream_t stream) {
  const AttnParams& p = sp.a;
  if (p.geom.dtype == PDA_BF16) {
    if (p.geom.head_dim == 128) return launch<128, false, 3, 4>(sp, stream);
    return launch<64, false, 3, 4>(sp, stream);
  }
  return launch<128, true, 3, 4>(sp, stream);
}

cudaError_t launch_attention_tma(const AttnParams& p, cudaStream_t stream) {
  const StepParams sp{p, nullptr, nullptr, nullptr, nullptr, nullptr, 0};
  return launch_step_tma(sp, stream);
}

}  // namespace pda
