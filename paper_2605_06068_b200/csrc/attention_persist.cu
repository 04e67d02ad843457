// Persistent fused decode step for unsplit launches (sm_100a): KV append + paged decode
// attention, one unit = (sequence, kv head), every unit written straight to `out`.
//
// The one-CTA-per-unit kernel (attention_tma.cu) pays a start-up chain per unit (sequence
// length -> block-table entries -> first TMA copy lands) during which the CTA's stages are
// empty. Here a fixed set of CTAs (as many as fit on the GPU) loops over the units instead:
//   * units are served longest first: every CTA ranks the sequences by length once (shared
//     memory) and an atomic ticket in the caller's workspace hands out (rank, kv head) pairs;
//   * the ticket of the NEXT unit is claimed late, when warp 0 has only a few tiles left, so
//     no CTA hoards work it will not reach for a long time (that ruins the tail);
//   * it is handed to the other warps through an mbarrier; each warp then loads the next unit's
//     page ids while it is still streaming, and as soon as it has consumed its last tile it
//     issues the next unit's first TMA copies: the per-warp stage ring never drains;
//   * the warps' (m, l, O) states are merged in registers through a small shared buffer (tree
//     over warps), so the ring stays free for those copies.
// The page pipeline and the tile math are those of attention_tma.cu (per-warp TMA rings,
// decode_tile). No CTA ever waits for another CTA; every mbarrier wait is bounded.
#include "common.cuh"
#include "decode_tile.cuh"
#include "tma_ptx.cuh"

namespace pda {

namespace {

constexpr int kMaxBatchPersist = 256;  // ranking is O(batch^2 / threads) per CTA
constexpr int kClaimLead = 3;          // tiles warp 0 still has to go when the next ticket is published

template <int D, bool kFp8, int kStages, int kWarps>
struct PersistCfg {
  static constexpr int kRowBytes = D * (kFp8 ? 1 : 2);
  static constexpr int kRowChunks = kRowBytes / 16;
  static constexpr int kTileBytes = kPageSize * kRowBytes;
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kWarpRing = kStages * kStageBytes;
  static constexpr int kKSteps = D / 16;
  static constexpr int kMergeFloats = kKSteps * 4 + 4;  // per lane: O fragment, m0, m1, l0, l1
  static constexpr int kMergeBytes = (kWarps / 2) * kMergeFloats * 32 * 4;
  static constexpr int kRingBytes = kWarps * kWarpRing;
  static constexpr int kBarBytes = (kWarps * kStages + 2) * 8;
  static constexpr int kTableBytes = 2 * kMaxBatchPersist * 4;  // order[B], lens[B]
  static constexpr int kMiscBytes = 64;
  static constexpr int kSmemBytes = kRingBytes + kMergeBytes + kBarBytes + kTableBytes + kMiscBytes + 1024;
  static_assert((kWarps & (kWarps - 1)) == 0 && kWarps >= 2, "tree merge needs a power of two");
};

__device__ __forceinline__ void mbar_arrive_p(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

struct Unit {
  int valid, b, g, L, n_tiles, err;
};

template <int D, bool kFp8, int kStages, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
attention_persist_kernel(const __grid_constant__ CUtensorMap k_map,
                         const __grid_constant__ CUtensorMap v_map, StepParams sp) {
  using C = PersistCfg<D, kFp8, kStages, kWarps>;
  const AttnParams& p = sp.a;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* merge_buf = reinterpret_cast<float*>(smem + C::kRingBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kRingBytes + C::kMergeBytes);
  int* order = reinterpret_cast<int*>(smem + C::kRingBytes + C::kMergeBytes + C::kBarBytes);  // rank -> sequence
  int* lens = order + kMaxBatchPersist;
  int* misc = lens + kMaxBatchPersist;  // [0] current ticket, [1] next ticket, [2] abort, [4..5] unit error
  constexpr int kThreads = kWarps * 32;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tq = lane & 3;
  const int B = p.batch, Hkv = p.geom.num_kv_heads, G = p.group;
  const int total_units = B * Hkv;
  int* ws = sp.workspace;

  // ---- set-up: barriers, lengths, ranking (longest first, ties by index)
  const uint32_t ring = smem_u32(smem + warp * C::kWarpRing);
  const uint32_t bar0 = smem_u32(bars + warp * kStages);
  const uint32_t bar_tk = smem_u32(bars + kWarps * kStages);
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
    if (warp == 0) mbar_init(bar_tk, 1);
    fence_mbar_init();
    fence_proxy_async();
  }
  if (tid < 8) misc[tid] = 0;
  // (one key per sequence, (length << 8) | (255 - index): distinct and larger for the sequence that comes
  // first; a rank is the number of larger keys, counted four keys to a load. The keys lie in the ring,
  // which no copy has been sent to yet. Lengths from 2^23 on rank as equal.)
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem);
  const int n_keys = (B + 3) & ~3;
  for (int j = tid; j < n_keys; j += kThreads) {
    const int Lj = j < B ? max(p.seq_lens[j], 0) : 0;
    if (j < B) lens[j] = Lj;
    keys[j] = j < B ? (static_cast<uint32_t>(min(Lj, (1 << 23) - 1)) << 8) | static_cast<uint32_t>(255 - j) : 0u;
  }
  __syncthreads();
  for (int j = tid; j < B; j += kThreads) {
    const uint32_t kj = keys[j];
    int rank = 0;
    for (int i = 0; i < n_keys; i += 4) {
      const uint4 k4 = *reinterpret_cast<const uint4*>(keys + i);
      rank += (k4.x > kj) + (k4.y > kj) + (k4.z > kj) + (k4.w > kj);
    }
    order[rank] = j;
  }
  if (tid == 0) misc[0] = atomicAdd(&ws[0], 1);
  __syncthreads();

  auto decode = [&](int T) -> Unit {
    Unit u;
    u.valid = T < total_units;
    u.b = u.g = u.L = u.n_tiles = u.err = 0;
    if (!u.valid) return u;
    u.g = T % Hkv;  // kv head fastest: the heads of one sequence share its pages
    u.b = order[T / Hkv];
    u.L = lens[u.b];
    if (static_cast<int64_t>(u.L) > static_cast<int64_t>(p.block_table_stride) * kPageSize)
      u.err = PDA_DEV_BAD_SEQ_LEN;
    u.n_tiles = u.err ? 0 : (u.L + kPageSize - 1) / kPageSize;
    return u;
  };
  auto tiles_of = [&](const Unit& u) { return u.n_tiles > warp ? (u.n_tiles - warp + kWarps - 1) / kWarps : 0; };
  // page ids (and e4m3 scales) of this warp's tiles of `u`, ordinals blk*32 .. blk*32+31; -1 marks a bad id
  auto load_block = [&](const Unit& u, int n_mine, int blk, int& pg, float& ks, float& vs) {
    const int kk = blk * 32 + lane;
    pg = 0; ks = 0.f; vs = 0.f;
    if (kk < n_mine) {
      const int v = p.block_table[static_cast<int64_t>(u.b) * p.block_table_stride + warp + kk * kWarps];
      pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
      if (kFp8) {
        ks = p.k_scale[static_cast<int64_t>(max(pg, 0)) * Hkv + u.g];
        vs = p.v_scale[static_cast<int64_t>(max(pg, 0)) * Hkv + u.g];
      }
    }
  };
  const uint32_t leader = elect_one();
  const uint64_t pol = l2_policy_evict_first();  // the tiles are read once: first out of the L2
  auto issue = [&](uint32_t ordinal, int g, int page_raw) {  // whole warp, converged; the elected lane issues
    const int s = ordinal % kStages;
    const uint32_t bar = bar0 + 8 * s;
    const uint32_t dst = ring + s * C::kStageBytes;
    mbar_expect_tx_if(leader, bar, C::kStageBytes);
    tma_load_5d_hint_if(leader, dst, &k_map, bar, 0, g, max(page_raw, 0), pol);
    tma_load_5d_hint_if(leader, dst + C::kTileBytes, &v_map, bar, 0, g, max(page_raw, 0), pol);
  };

  const float scale_log2 = p.scale * 1.4426950408889634f;
  uint32_t ord = 0;        // tiles this warp has consumed so far (ring position)
  bool bad_page = false;   // warp-uniform: a page id of the unit being streamed was out of range
  Unit cur = decode(misc[0]);
  int n_mine = tiles_of(cur);
  int pgA, pgB, pgN = 0;
  float ksA, ksB, vsA, vsB, ksN = 0.f, vsN = 0.f;
  load_block(cur, n_mine, 0, pgA, ksA, vsA);
  for (int j = 0; j < min(kStages, n_mine); ++j) {
    const int page = __shfl_sync(0xffffffffu, pgA, j);
    if (page < 0) bad_page = true;
    issue(ord + j, cur.g, page);
  }

  // Q^T fragments of the current unit and, once its ticket is known, of the next one
  uint32_t qf[C::kKSteps][2], qfN[C::kKSteps][2];
  if (cur.valid)
    load_q_fragments<D, kFp8>(p.q + (static_cast<int64_t>(cur.b) * p.num_q_heads + static_cast<int64_t>(cur.g) * G) * D,
                              G, gid, tq, qf);
#pragma unroll
  for (int i = 0; i < C::kKSteps; ++i) { qfN[i][0] = 0u; qfN[i][1] = 0u; }

  for (int iter = 0; cur.valid; ++iter) {
    const uint32_t tk_parity = iter & 1;
    const int64_t row0 = static_cast<int64_t>(cur.b) * p.num_q_heads + static_cast<int64_t>(cur.g) * G;
    pgB = 0; ksB = 0.f; vsB = 0.f;
    if (n_mine > 32) load_block(cur, n_mine, 1, pgB, ksB, vsB);  // only long units need a second block
    const bool append_here = sp.k_new != nullptr && !cur.err && cur.L > 0;

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // heads 2tq, 2tq+1
    float o[C::kKSteps][4];
#pragma unroll
    for (int i = 0; i < C::kKSteps; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

    // the next unit: claimed late by thread 0, picked up by every warp while it still streams
    int tk_reg = 0;
    bool claim_issued = false, claim_published = false;  // thread 0 only
    Unit nxt;
    nxt.valid = 0; nxt.b = nxt.g = nxt.L = nxt.n_tiles = nxt.err = 0;
    int n_next = 0;
    bool have_next = false;

    bool timed_out = false;
    int kk = 0;
    for (; kk < n_mine; ++kk) {
      const int remaining = n_mine - kk;
      if (tid == 0) {
        if (claim_issued && !claim_published && remaining <= kClaimLead) {
          misc[1] = tk_reg;
          mbar_arrive_p(bar_tk);
          claim_published = true;
        }
        if (!claim_issued && remaining <= kClaimLead + 1) {
          tk_reg = atomicAdd(&ws[0], 1);  // consumed one tile later: the round trip is off the critical path
          claim_issued = true;
        }
      }
      if (!have_next && remaining < kClaimLead) {
        const bool ready = __all_sync(0xffffffffu, mbar_test_wait(bar_tk, tk_parity));
        if (ready) {
          nxt = decode(misc[1]);
          n_next = tiles_of(nxt);
          load_block(nxt, n_next, 0, pgN, ksN, vsN);
          if (nxt.valid)
            load_q_fragments<D, kFp8>(p.q + (static_cast<int64_t>(nxt.b) * p.num_q_heads +
                                             static_cast<int64_t>(nxt.g) * G) * D, G, gid, tq, qfN);
          have_next = true;
        }
      }

      const uint32_t ordinal = ord + kk;
      const int s = ordinal % kStages;
      if (!mbar_wait_bounded(bar0 + 8 * s, (ordinal / kStages) & 1)) { timed_out = true; break; }
      const uint32_t kt = ring + s * C::kStageBytes, vt = kt + C::kTileBytes;
      const int tile = warp + kk * kWarps;
      const int n_valid = min(kPageSize, cur.L - tile * kPageSize);
      float ksc = 1.f, vsc = 1.f;
      if (kFp8) {
        ksc = __shfl_sync(0xffffffffu, ksA, kk & 31);
        vsc = __shfl_sync(0xffffffffu, vsA, kk & 31);
      }
      if (!kFp8 && append_here && tile == cur.n_tiles - 1) {
        // fused append: the new token's K/V rows go into the landed tile and into the cache
        const int slot = (cur.L - 1) % kPageSize;
        const int page = __shfl_sync(0xffffffffu, pgA, kk & 31);
        if (lane < C::kRowChunks && page >= 0) {
          const int64_t src = (static_cast<int64_t>(cur.b) * Hkv + cur.g) * D + lane * 8;
          const uint4 kv = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.k_new) + src);
          const uint4 vv = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(sp.v_new) + src);
          const int64_t dst = page * p.geom.page_stride + cur.g * p.geom.head_stride +
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

      decode_tile<D, kFp8>(kt, vt, n_valid, 0, scale_log2 * ksc, vsc, qf, m0, m1, l0, l1, o, lane);

      // ---- hand the stage back and refill it
      __syncwarp();
      const int kn = kk + kStages;
      if (((kk + 1) & 31) == 0) {
        pgA = pgB; ksA = ksB; vsA = vsB;
        load_block(cur, n_mine, (kk + 1) / 32 + 1, pgB, ksB, vsB);
      }
      if (kn < n_mine) {
        // (a branch, not a select: block B's loads must not be waited for while block A serves)
        int page;
        if ((kn >> 5) == ((kk + 1) >> 5)) page = __shfl_sync(0xffffffffu, pgA, kn & 31);
        else page = __shfl_sync(0xffffffffu, pgB, kn & 31);
        if (page < 0) bad_page = true;
        fence_proxy_async();
        issue(ord + kn, cur.g, page);
      }
    }

    if (timed_out) {
      for (int j = kk; j < min(kk + kStages, n_mine); ++j)
        mbar_wait_bounded(bar0 + 8 * ((ord + j) % kStages), ((ord + j) / kStages) & 1);
      if (lane == 0) atomicMax(&misc[2], PDA_DEV_TIMEOUT);
    }
    ord += n_mine;
    int* unit_err_slot = &misc[4 + (iter & 1)];
    if (bad_page && lane == 0) atomicMax(unit_err_slot, PDA_DEV_BAD_PAGE);
    if (timed_out && lane == 0) atomicMax(unit_err_slot, PDA_DEV_TIMEOUT);
    bad_page = false;

    // ---- the next unit, for warps that have not seen its ticket yet
    if (tid == 0) {
      if (!claim_issued) tk_reg = atomicAdd(&ws[0], 1);
      if (!claim_published) {
        misc[1] = tk_reg;
        mbar_arrive_p(bar_tk);
      }
      misc[4 + ((iter + 1) & 1)] = 0;  // the next unit's error slot (last read before this unit began)
    }
    if (!have_next) {
      const bool ready = __all_sync(0xffffffffu, mbar_wait_bounded(bar_tk, tk_parity));
      if (ready) {
        nxt = decode(misc[1]);
        n_next = tiles_of(nxt);
        load_block(nxt, n_next, 0, pgN, ksN, vsN);
        if (nxt.valid)
          load_q_fragments<D, kFp8>(p.q + (static_cast<int64_t>(nxt.b) * p.num_q_heads +
                                           static_cast<int64_t>(nxt.g) * G) * D, G, gid, tq, qfN);
      } else if (lane == 0) {
        atomicMax(&misc[2], PDA_DEV_TIMEOUT);
      }
    }
    // ---- keep the ring busy: first tiles of the next unit
    int n_prefetched = 0;
    if (!timed_out && nxt.valid) {
      n_prefetched = min(kStages, n_next);
      for (int j = 0; j < n_prefetched; ++j) {
        const int page = __shfl_sync(0xffffffffu, pgN, j);
        if (page < 0) bad_page = true;  // belongs to the next unit: reported when that unit ends
        if (lane == 0) {
          if (j == 0) fence_proxy_async();
          issue(ord + j, nxt.g, page);
        }
      }
    }

    // ---- merge the warps' states in registers (tree over warps through merge_buf)
#pragma unroll
    for (int half = kWarps / 2; half >= 1; half >>= 1) {
      if (warp >= half && warp < 2 * half) {
        float* dst = merge_buf + (warp - half) * C::kMergeFloats * 32 + lane;
#pragma unroll
        for (int mt = 0; mt < C::kKSteps; ++mt)
#pragma unroll
          for (int e = 0; e < 4; ++e) dst[(mt * 4 + e) * 32] = o[mt][e];
        dst[(C::kKSteps * 4 + 0) * 32] = m0; dst[(C::kKSteps * 4 + 1) * 32] = m1;
        dst[(C::kKSteps * 4 + 2) * 32] = l0; dst[(C::kKSteps * 4 + 3) * 32] = l1;
      }
      __syncthreads();
      if (warp < half) {
        const float* src = merge_buf + warp * C::kMergeFloats * 32 + lane;
        const float om0 = src[(C::kKSteps * 4 + 0) * 32], om1 = src[(C::kKSteps * 4 + 1) * 32];
        const float ol0 = src[(C::kKSteps * 4 + 2) * 32], ol1 = src[(C::kKSteps * 4 + 3) * 32];
        const float M0 = fmaxf(m0, om0), M1 = fmaxf(m1, om1);
        const float a0 = m0 > -INFINITY ? ex2(m0 - M0) : 0.f, b0 = om0 > -INFINITY ? ex2(om0 - M0) : 0.f;
        const float a1 = m1 > -INFINITY ? ex2(m1 - M1) : 0.f, b1 = om1 > -INFINITY ? ex2(om1 - M1) : 0.f;
        m0 = M0; m1 = M1;
        l0 = l0 * a0 + ol0 * b0;
        l1 = l1 * a1 + ol1 * b1;
#pragma unroll
        for (int mt = 0; mt < C::kKSteps; ++mt) {
          o[mt][0] = o[mt][0] * a0 + src[(mt * 4 + 0) * 32] * b0;
          o[mt][1] = o[mt][1] * a1 + src[(mt * 4 + 1) * 32] * b1;
          o[mt][2] = o[mt][2] * a0 + src[(mt * 4 + 2) * 32] * b0;
          o[mt][3] = o[mt][3] * a1 + src[(mt * 4 + 3) * 32] * b1;
        }
      }
      __syncthreads();
    }

    // ---- warp 0 writes the unit's output rows
    if (warp == 0) {
      const int unit_err = max(max(cur.err, *unit_err_slot), misc[2]);  // stable: written before the merge barriers
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
      }
      const bool live0 = !unit_err && l0 > 0.f, live1 = !unit_err && l1 > 0.f;
      const float inv0 = live0 ? 1.f / l0 : 0.f, inv1 = live1 ? 1.f / l1 : 0.f;
      const int h0 = 2 * tq, h1 = 2 * tq + 1;
#pragma unroll
      for (int mt = 0; mt < C::kKSteps; ++mt) {
        const int d0 = kFp8 ? 16 * mt + 2 * gid : 16 * mt + gid;
        const int d1 = kFp8 ? d0 + 1 : d0 + 8;
        if (h0 < G) {
          p.out[(row0 + h0) * D + d0] = __float2bfloat16_rn(live0 ? o[mt][0] * inv0 : 0.f);
          p.out[(row0 + h0) * D + d1] = __float2bfloat16_rn(live0 ? o[mt][2] * inv0 : 0.f);
        }
        if (h1 < G) {
          p.out[(row0 + h1) * D + d0] = __float2bfloat16_rn(live1 ? o[mt][1] * inv1 : 0.f);
          p.out[(row0 + h1) * D + d1] = __float2bfloat16_rn(live1 ? o[mt][3] * inv1 : 0.f);
        }
      }
      if (unit_err && lane == 0) report(p.status, unit_err);
    }
    __syncthreads();  // merge_buf, the ticket slot and the error slots may be reused from here on

    if (misc[2] == PDA_DEV_TIMEOUT) {  // a wait expired: stop taking work, drain what is in flight
      for (int j = 0; j < n_prefetched; ++j)
        mbar_wait_bounded(bar0 + 8 * ((ord + j) % kStages), ((ord + j) / kStages) & 1);
      break;
    }
    cur = nxt;
    n_mine = n_next;
    pgA = pgN; ksA = ksN; vsA = vsN;
#pragma unroll
    for (int i = 0; i < C::kKSteps; ++i) { qf[i][0] = qfN[i][0]; qf[i][1] = qfN[i][1]; }
  }

  // ---- the last CTA out re-arms the ticket counter for the next launch
  if (tid == 0) {
    const int prev = atomicAdd(&ws[1], 1);
    if (prev == static_cast<int>(gridDim.x) - 1) {
      ws[0] = 0;
      ws[1] = 0;
    }
  }
}

template <int D, bool kFp8, int kStages, int kWarps>
cudaError_t launch(const StepParams& sp, cudaStream_t stream) {
  using C = PersistCfg<D, kFp8, kStages, kWarps>;
  const AttnParams& p = sp.a;
  alignas(64) CUtensorMap k_map, v_map;
  const int eb = p.geom.dtype == PDA_BF16 ? 2 : 1;
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb))
    return cudaErrorNotSupported;
  auto kern = attention_persist_kernel<D, kFp8, kStages, kWarps>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  // resident CTAs: as many as the device holds at once (cached per device)
  static int cached_grid[64] = {};
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (cached_grid[dev] == 0) {
    int sms = 0, per_sm = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kWarps * 32, C::kSmemBytes)) != cudaSuccess)
      return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    cached_grid[dev] = sms * per_sm;
  }
  const int64_t units = static_cast<int64_t>(p.batch) * p.geom.num_kv_heads;
  const unsigned grid = static_cast<unsigned>(units < cached_grid[dev] ? units : cached_grid[dev]);
  kern<<<grid, kWarps * 32, C::kSmemBytes, stream>>>(k_map, v_map, sp);
  return cudaGetLastError();
}

}  // namespace

bool attention_persist_supports(const StepParams& sp) {
  const AttnParams& p = sp.a;
  return attention_tma_supports(p) && sp.workspace != nullptr && p.chunk_tokens == 0 && p.window == 0 &&
         p.first_token == 0 && p.batch <= kMaxBatchPersist && p.batch >= 1;
}

// The persistent loop pays barriers per unit that a fresh CTA does not; it wins once every
// resident CTA serves many (short) units, so that the start-up chain it hides dominates.
// Measured on B200: chat70b (2048 units, 6.9 per resident CTA) 224 vs 239 us; llama8b (512
// units, 1.7 per CTA) 104-108 vs 100 us; prefix_fp8 (1024 units, 3.5 per CTA) 126 vs 101 us.
bool attention_persist_preferred(const StepParams& sp, int min_units_per_cta) {
  static int sms_cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (sms_cached[dev] == 0 &&
      cudaDeviceGetAttribute(&sms_cached[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return false;
  const int64_t units = static_cast<int64_t>(sp.a.batch) * sp.a.geom.num_kv_heads;
  return units >= static_cast<int64_t>(min_units_per_cta) * 2 * sms_cached[dev];  // 2 CTAs per SM
}

cudaError_t launch_attention_persist(const StepParams& sp, cudaStream_t stream) {
  const AttnParams& p = sp.a;
  if (p.geom.dtype == PDA_BF16) {
    if (p.geom.head_dim == 128) return launch<128, false, 3, 4>(sp, stream);
    return launch<64, false, 3, 4>(sp, stream);
  }
  return launch<128, true, 3, 4>(sp, stream);
}

}  // namespace pda
