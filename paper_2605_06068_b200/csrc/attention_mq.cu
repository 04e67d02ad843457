// Multi-query paged attention for sm_100a: many query rows against one
// sequence's paged KV, as dense tensor-core tiles. Two uses:
//   * verification of a block of T draft tokens (n_q = T, causal inside the
//     block): rows = T x G per (sequence, kv head);
//   * the shared-prefix part of a decode batch (n_q = number of sequences that
//     share the prefix, not causal): rows = B x G per kv head, computed once
//     instead of once per sequence.
// Here the query rows are the M dimension (16 per warp), so QK^T and PV are the
// classic flash-attention tiles: S[16 x 16] = Q[16 x D] . K_page^T, row-wise
// online softmax, O[16 x D] += P[16 x 16] . V_page, with the S accumulator
// registers reused directly as the A operand of PV.
//
// CTA = one producer warp + kConsumers consumer warps (16 rows each) working on
// (row block, kv head, sequence, chunk). The producer streams (K tile, V tile)
// page stages through a CTA-wide ring with 5-D tiled TMA copies (full barriers
// by transaction bytes, empty barriers by one arrival per consumer warp); every
// consumer warp reads every stage, so a page is fetched once for up to 128 rows.
// e4m3 pages are converted to f16 in registers; per-(page, head) scales travel
// with the stage. All waits are bounded. No multicast.
#include "common.cuh"
#include "tma_ptx.cuh"

namespace pda {

namespace {

template <int D, bool kFp8, int kStages, int kConsumers>
struct MqCfg {
  static constexpr int kElem = kFp8 ? 1 : 2;
  static constexpr int kRowBytes = D * kElem;
  static constexpr int kTileBytes = kPageSize * kRowBytes;
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kKSteps = D / 16;
  static constexpr int kThreads = (kConsumers + 1) * 32;
  static constexpr int kRows = kConsumers * 16;
  static constexpr int kRingBytes = kStages * kStageBytes;
  static constexpr int kSmemBytes = kRingBytes + kStages * (8 + 8 + 8) + 32 + 1024;
  static_assert(kRowBytes % 128 == 0, "rows must be whole 128-byte swizzle lines");
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int D, bool kFp8, int kStages, int kConsumers>
__global__ void __launch_bounds__((kConsumers + 1) * 32)
attention_mq_kernel(const __grid_constant__ CUtensorMap k_map,
                    const __grid_constant__ CUtensorMap v_map, MqParams mp) {
  using C = MqCfg<D, kFp8, kStages, kConsumers>;
  const AttnParams& p = mp.a;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::kRingBytes);
  uint64_t* empty = full + kStages;
  float* stage_scales = reinterpret_cast<float*>(empty + kStages);  // [kStages][2]: k_scale, v_scale
  int* cta_err = reinterpret_cast<int*>(stage_scales + 2 * kStages);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tq = lane & 3;
  const int G = p.group, T = mp.n_q;
  const int rows_total = T * G;
  const int n_rb = (rows_total + C::kRows - 1) / C::kRows;
  const int c = blockIdx.x, g = blockIdx.y / n_rb, rb = blockIdx.y % n_rb, b = blockIdx.z;
  const bool split = p.chunk_tokens > 0;

  const int L = mp.kv_len_fixed > 0 ? mp.kv_len_fixed : max(p.seq_lens[b], 0);
  int t0 = p.first_token, t1 = L;
  if (split) {
    t0 = p.first_token + c * p.chunk_tokens;
    if (t0 >= L) return;
    t1 = min(t0 + p.chunk_tokens, L);
  }
  int err = 0;
  if (static_cast<int64_t>(L) > static_cast<int64_t>(p.block_table_stride) * kPageSize ||
      (split && static_cast<int64_t>(L - p.first_token) >
                    static_cast<int64_t>(p.max_chunks - p.chunk_slot0) * p.chunk_tokens))
    err = PDA_DEV_BAD_SEQ_LEN;
  const int page0 = t0 / kPageSize;
  const int n_tiles = err ? 0 : (t1 + kPageSize - 1) / kPageSize - page0;

  const uint32_t ring = smem_u32(smem);
  const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty);
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kConsumers);
    }
    *cta_err = 0;
    fence_mbar_init();
    fence_proxy_async();
  }
  __syncthreads();

  const int32_t* table = p.block_table + static_cast<int64_t>(b) * p.block_table_stride;

  if (warp == kConsumers) {
    // ================= producer warp =================
    const uint32_t leader = elect_one();
    bool bad = false;
    int pg = 0;
    for (int i = 0; i < n_tiles; ++i) {
      if ((i & 31) == 0) {  // page ids of the next 32 tiles, one per lane
        pg = 0;
        if (i + lane < n_tiles) {
          const int v = table[page0 + i + lane];
          pg = (v < 0 || v >= p.geom.num_pages) ? -1 : v;
        }
      }
      const int page_raw = __shfl_sync(0xffffffffu, pg, i & 31);
      if (page_raw < 0) bad = true;
      const int page = max(page_raw, 0);
      const int s = i % kStages;
      bool ok = true;
      if (i >= kStages) ok = mbar_wait_bounded(empty0 + 8 * s, ((i / kStages) - 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); break; }
      if (kFp8 && lane == 0) {
        stage_scales[2 * s] = p.k_scale[static_cast<int64_t>(page) * p.geom.num_kv_heads + g];
        stage_scales[2 * s + 1] = p.v_scale[static_cast<int64_t>(page) * p.geom.num_kv_heads + g];
      }
      __syncwarp();
      const uint32_t dst = ring + s * C::kStageBytes;
      fence_proxy_async();
      // (the elected lane issues, predicated: see elect_one)
      mbar_expect_tx_if(leader, full0 + 8 * s, C::kStageBytes);
      tma_load_5d_if(leader, dst, &k_map, full0 + 8 * s, 0, g, page);
      tma_load_5d_if(leader, dst + C::kTileBytes, &v_map, full0 + 8 * s, 0, g, page);
    }
    if (bad && lane == 0) atomicMax(cta_err, PDA_DEV_BAD_PAGE);
  }

  // ================= consumer warps =================
  // rows of this warp: local row r -> (query token i = r / G, head of the group hh = r % G)
  const int r_lo = rb * C::kRows + warp * 16 + gid, r_hi = r_lo + 8;
  const bool consumer = warp < kConsumers;
  const bool v_lo = consumer && r_lo < rows_total, v_hi = consumer && r_hi < rows_total;
  const int i_lo = r_lo / G, i_hi = r_hi / G;
  const int64_t qrow_lo = (static_cast<int64_t>(b) * T + i_lo) * p.num_q_heads + g * G + (r_lo % G);
  const int64_t qrow_hi = (static_cast<int64_t>(b) * T + i_hi) * p.num_q_heads + g * G + (r_hi % G);
  // keys visible to a row: [first attended token, limit)
  const int lim_lo = mp.causal ? min(L, L - T + i_lo + 1) : L;
  const int lim_hi = mp.causal ? min(L, L - T + i_hi + 1) : L;

  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  float o[2 * C::kKSteps][4];  // 16 x D accumulator: n-tile j covers 8 output columns
#pragma unroll
  for (int j = 0; j < 2 * C::kKSteps; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

  if (consumer) {
    // ---- Q fragments (A operand), resident for the whole unit
    uint32_t qf[C::kKSteps][4];
    {
      const __nv_bfloat16* ql = p.q + qrow_lo * D;
      const __nv_bfloat16* qh = p.q + qrow_hi * D;
#pragma unroll
      for (int ks = 0; ks < C::kKSteps; ++ks) {
        qf[ks][0] = qf[ks][1] = qf[ks][2] = qf[ks][3] = 0u;
        if (!kFp8) {
          if (v_lo) {
            qf[ks][0] = *reinterpret_cast<const uint32_t*>(ql + 16 * ks + 2 * tq);
            qf[ks][2] = *reinterpret_cast<const uint32_t*>(ql + 16 * ks + 2 * tq + 8);
          }
          if (v_hi) {
            qf[ks][1] = *reinterpret_cast<const uint32_t*>(qh + 16 * ks + 2 * tq);
            qf[ks][3] = *reinterpret_cast<const uint32_t*>(qh + 16 * ks + 2 * tq + 8);
          }
        } else {
          // e4m3 K fragments put d = 16ks+4tq+{0,1} in k-slots {2tq,2tq+1} and d = 16ks+4tq+{2,3}
          // in k-slots {2tq+8,2tq+9}; q is loaded in the same order and converted to f16
          if (v_lo) {
            const uint2 raw = *reinterpret_cast<const uint2*>(ql + 16 * ks + 4 * tq);
            qf[ks][0] = pack2<true>(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u));
            qf[ks][2] = pack2<true>(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
          }
          if (v_hi) {
            const uint2 raw = *reinterpret_cast<const uint2*>(qh + 16 * ks + 4 * tq);
            qf[ks][1] = pack2<true>(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u));
            qf[ks][3] = pack2<true>(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
          }
        }
      }
    }

    const float scale_log2 = p.scale * 1.4426950408889634f;
    const int lj = lane >> 3, lr = lane & 7;
    // K as B operand (ldmatrix, not transposed): matrices (tok 0-7, chunk c0), (tok 0-7, c0+1),
    // (tok 8-15, c0), (tok 8-15, c0+1) -> b0,b1 of token tile 0 and b0,b1 of token tile 1.
    // For e4m3 one 16-byte chunk is a whole k-step: (tok 0-7, c), (tok 8-15, c), (.., c+1), (.., c+1).
    const int kb_row = kFp8 ? lr + 8 * (lj & 1) : lr + 8 * (lj >> 1);
    const int kb_chk = kFp8 ? (lj >> 1) : (lj & 1);
    // V as B operand (ldmatrix.trans): matrices (tok 0-7, chunk c0), (tok 8-15, c0), (tok 0-7, c0+1),
    // (tok 8-15, c0+1) -> b0,b1 of output tile c0 and of output tile c0+1.
    const int vb_row = lr + 8 * (lj & 1), vb_chk = lj >> 1;

    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kStages;
      bool ok = mbar_wait_bounded(full0 + 8 * s, (i / kStages) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { if (lane == 0) atomicMax(cta_err, PDA_DEV_TIMEOUT); break; }
      const uint32_t kt = ring + s * C::kStageBytes, vt = kt + C::kTileBytes;
      const int tok0 = (page0 + i) * kPageSize;
      float ksc = 1.f, vsc = 1.f;
      if (kFp8) { ksc = stage_scales[2 * s]; vsc = stage_scales[2 * s + 1]; }

      // ---- S = Q . K^T : two 8-token column tiles
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
      if (!kFp8) {
#pragma unroll
        for (int ks = 0; ks < C::kKSteps; ++ks) {
          uint32_t r[4];
          ldsm_x4(kt + tile_off(kb_row, 2 * ks + kb_chk), r);
          mma16816<false>(s0, qf[ks], r[0], r[1]);
          mma16816<false>(s1, qf[ks], r[2], r[3]);
        }
      } else {
#pragma unroll
        for (int ks = 0; ks < C::kKSteps; ks += 2) {
          uint32_t r[4];
          ldsm_x4(kt + tile_off(kb_row, ks + kb_chk), r);  // r0: tok 0-7 chunk ks, r1: tok 8-15 chunk ks, r2/r3: chunk ks+1
          uint32_t c[4][2];
#pragma unroll
          for (int i = 0; i < 4; ++i) e4m3x4_to_f16x2x2(r[i], c[i][0], c[i][1]);
          mma16816<true>(s0, qf[ks], c[0][0], c[0][1]);
          mma16816<true>(s1, qf[ks], c[1][0], c[1][1]);
          mma16816<true>(s0, qf[ks + 1], c[2][0], c[2][1]);
          mma16816<true>(s1, qf[ks + 1], c[3][0], c[3][1]);
        }
      }
      const float sc = scale_log2 * ksc;
      // accumulator layout: [0],[1] = row gid, cols 2tq,2tq+1 ; [2],[3] = row gid+8
#pragma unroll
      for (int e = 0; e < 4; ++e) { s0[e] *= sc; s1[e] *= sc; }
      if (tok0 + kPageSize > min(lim_lo, lim_hi)) {  // (chunk starts are page-aligned: no lower cut)
        const int c0 = tok0 + 2 * tq, c1 = c0 + 1, c8 = c0 + 8, c9 = c0 + 9;
        if (c0 >= lim_lo) s0[0] = -INFINITY;
        if (c1 >= lim_lo) s0[1] = -INFINITY;
        if (c8 >= lim_lo) s1[0] = -INFINITY;
        if (c9 >= lim_lo) s1[1] = -INFINITY;
        if (c0 >= lim_hi) s0[2] = -INFINITY;
        if (c1 >= lim_hi) s0[3] = -INFINITY;
        if (c8 >= lim_hi) s1[2] = -INFINITY;
        if (c9 >= lim_hi) s1[3] = -INFINITY;
      }

      // ---- row-wise online softmax (base 2); a row may have no visible key in this tile
      float mx_lo = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
      float mx_hi = fmaxf(fmaxf(s0[2], s0[3]), fmaxf(s1[2], s1[3]));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float ref_lo = mn_lo == -INFINITY ? 0.f : mn_lo, ref_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const float al_lo = ex2(m_lo - ref_lo), al_hi = ex2(m_hi - ref_hi);
      m_lo = mn_lo; m_hi = mn_hi;
      const float p00 = ex2(s0[0] - ref_lo), p01 = ex2(s0[1] - ref_lo), p10 = ex2(s1[0] - ref_lo), p11 = ex2(s1[1] - ref_lo);
      const float p02 = ex2(s0[2] - ref_hi), p03 = ex2(s0[3] - ref_hi), p12 = ex2(s1[2] - ref_hi), p13 = ex2(s1[3] - ref_hi);
      l_lo = fmaf(l_lo, al_lo, (p00 + p01) + (p10 + p11));
      l_hi = fmaf(l_hi, al_hi, (p02 + p03) + (p12 + p13));
      // P as the A operand of PV: a0 = (row gid, tok 2tq..), a1 = (row gid+8, ..), a2/a3 = tokens +8
      uint32_t pa[4];
      pa[0] = pack2<kFp8>(p00 * vsc, p01 * vsc);
      pa[1] = pack2<kFp8>(p02 * vsc, p03 * vsc);
      pa[2] = pack2<kFp8>(p10 * vsc, p11 * vsc);
      pa[3] = pack2<kFp8>(p12 * vsc, p13 * vsc);

      // ---- O = O * alpha + P . V
#pragma unroll
      for (int j = 0; j < 2 * C::kKSteps; ++j) {
        o[j][0] *= al_lo; o[j][1] *= al_lo; o[j][2] *= al_hi; o[j][3] *= al_hi;
      }
      // keys past the end of the sequence may hold anything: clear them in the V fragments
      const int n_valid = L - tok0;  // >= 16 except in the sequence's last tile
      uint32_t keep0 = 0xffffffffu, keep1 = 0xffffffffu;  // tokens (2tq, 2tq+1) and (2tq+8, 2tq+9)
      if (n_valid < kPageSize) {
        keep0 = (2 * tq + 1 < n_valid) ? 0xffffffffu : (2 * tq < n_valid ? 0x0000ffffu : 0u);
        keep1 = (2 * tq + 9 < n_valid) ? 0xffffffffu : (2 * tq + 8 < n_valid ? 0x0000ffffu : 0u);
      }
      if (!kFp8) {
#pragma unroll
        for (int j = 0; j < C::kKSteps; ++j) {  // output tiles 2j, 2j+1 (d = 16j .. 16j+15)
          uint32_t r[4];
          ldsm_x4_trans(vt + tile_off(vb_row, 2 * j + vb_chk), r);
          mma16816<false>(o[2 * j], pa, r[0] & keep0, r[1] & keep1);
          mma16816<false>(o[2 * j + 1], pa, r[2] & keep0, r[3] & keep1);
        }
      } else {
#pragma unroll
        for (int j = 0; j < C::kKSteps; j += 2) {  // 16-byte chunks j, j+1 = d 16j .. 16j+31
          uint32_t r[4];
          ldsm_x4_trans(vt + tile_off(vb_row, j + vb_chk), r);
          // a transposed register holds bytes V[2tq][dA], V[2tq][dA+1], V[2tq+1][dA], V[2tq+1][dA+1],
          // dA = 16*chunk + 2gid: regroup into (V[2tq][d], V[2tq+1][d]) for d = dA (low) and dA+1 (high)
#pragma unroll
          for (int e = 0; e < 4; ++e) r[e] = __byte_perm(r[e], 0, 0x3120);
          // output tile 2j: columns n <-> d = 16j + 2n ; tile 2j+1: d = 16j + 2n + 1 (and likewise for chunk j+1)
          uint32_t c[4][2];
#pragma unroll
          for (int i = 0; i < 4; ++i) e4m3x4_to_f16x2x2(r[i], c[i][0], c[i][1]);
          mma16816<true>(o[2 * j], pa, c[0][0] & keep0, c[1][0] & keep1);
          mma16816<true>(o[2 * j + 1], pa, c[0][1] & keep0, c[1][1] & keep1);
          mma16816<true>(o[2 * j + 2], pa, c[2][0] & keep0, c[3][0] & keep1);
          mma16816<true>(o[2 * j + 3], pa, c[2][1] & keep0, c[3][1] & keep1);
        }
      }

      // ---- this warp is done with the stage
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
  }
  __syncthreads();

  // ---- finalise: each consumer thread owns 2 rows x (D/4) columns
  const int dev_err = max(err, *cta_err);
  if (dev_err && tid == 0) report(p.status, dev_err);
  if (consumer) {
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    constexpr float kLn2 = 0.6931471805599453f;
    const bool live_lo = !dev_err && l_lo > 0.f, live_hi = !dev_err && l_hi > 0.f;
    const float inv_lo = live_lo ? 1.f / l_lo : 0.f, inv_hi = live_hi ? 1.f / l_hi : 0.f;
#pragma unroll
    for (int j = 0; j < 2 * C::kKSteps; ++j) {
      // columns of accumulator tile j held by this thread
      int d0, d1;
      if (!kFp8) { d0 = 8 * j + 2 * tq; d1 = d0 + 1; }
      else { d0 = 16 * (j >> 1) + 4 * tq + (j & 1); d1 = d0 + 2; }
      if (split) {
        const int64_t slot = p.chunk_slot0 + c;
        if (v_lo) {
          float* dst = p.part_o + (qrow_lo * p.max_chunks + slot) * D;
          dst[d0] = o[j][0] * inv_lo; dst[d1] = o[j][1] * inv_lo;
        }
        if (v_hi) {
          float* dst = p.part_o + (qrow_hi * p.max_chunks + slot) * D;
          dst[d0] = o[j][2] * inv_hi; dst[d1] = o[j][3] * inv_hi;
        }
      } else {
        if (v_lo) {
          p.out[qrow_lo * D + d0] = __float2bfloat16_rn(o[j][0] * inv_lo);
          p.out[qrow_lo * D + d1] = __float2bfloat16_rn(o[j][1] * inv_lo);
        }
        if (v_hi) {
          p.out[qrow_hi * D + d0] = __float2bfloat16_rn(o[j][2] * inv_hi);
          p.out[qrow_hi * D + d1] = __float2bfloat16_rn(o[j][3] * inv_hi);
        }
      }
    }
    if (split && tq == 0) {
      const int64_t slot = p.chunk_slot0 + c;
      if (v_lo) p.part_lse[qrow_lo * p.max_chunks + slot] = live_lo ? (m_lo + __log2f(l_lo)) * kLn2 : -INFINITY;
      if (v_hi) p.part_lse[qrow_hi * p.max_chunks + slot] = live_hi ? (m_hi + __log2f(l_hi)) * kLn2 : -INFINITY;
    }
  }
}

template <int D, bool kFp8, int kStages, int kConsumers>
cudaError_t launch(const MqParams& mp, cudaStream_t stream) {
  using C = MqCfg<D, kFp8, kStages, kConsumers>;
  const AttnParams& p = mp.a;
  alignas(64) CUtensorMap k_map, v_map;
  const int eb = p.geom.dtype == PDA_BF16 ? 2 : 1;
  if (!make_cache_tensor_map(&k_map, p.k_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb) ||
      !make_cache_tensor_map(&v_map, p.v_cache, p.geom.page_stride, p.geom.head_stride, p.geom.slot_stride,
                             p.geom.num_pages, p.geom.num_kv_heads, p.geom.head_dim, eb))
    return cudaErrorNotSupported;
  auto kern = attention_mq_kernel<D, kFp8, kStages, kConsumers>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int rows_total = mp.n_q * p.group;
  const int n_rb = (rows_total + C::kRows - 1) / C::kRows;
  const unsigned chunks = p.chunk_tokens > 0 ? static_cast<unsigned>(mp.n_chunks_grid) : 1u;
  dim3 grid(chunks, p.geom.num_kv_heads * n_rb, p.batch);
  kern<<<grid, C::kThreads, C::kSmemBytes, stream>>>(k_map, v_map, mp);
  return cudaGetLastError();
}

}  // namespace

bool attention_mq_supports(const MqParams& mp) {
  const AttnParams& p = mp.a;
  if (p.group < 1 || mp.n_q < 1) return false;
  if (p.geom.head_dim != 128 && !(p.geom.head_dim == 64 && p.geom.dtype == PDA_BF16)) return false;
  const int64_t rows = static_cast<int64_t>(mp.n_q) * p.group;
  const int64_t n_rb = (rows + 63) / 64;
  return p.geom.num_kv_heads * n_rb <= 65535 && p.geom.num_pages >= 1;
}

cudaError_t launch_attention_mq(const MqParams& mp, cudaStream_t stream) {
  const AttnParams& p = mp.a;
  const int rows = mp.n_q * p.group;
  if (p.geom.dtype == PDA_BF16) {
    if (p.geom.head_dim == 128)
      return rows > 64 ? launch<128, false, 8, 8>(mp, stream) : launch<128, false, 8, 4>(mp, stream);
    return rows > 64 ? launch<64, false, 8, 8>(mp, stream) : launch<64, false, 8, 4>(mp, stream);
  }
  return rows > 64 ? launch<128, true, 12, 8>(mp, stream) : launch<128, true, 12, 4>(mp, stream);
}

}  // namespace pda
