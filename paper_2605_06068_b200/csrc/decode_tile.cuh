// The per-page tile of decode attention, shared by the decode kernels: for one landed
// (K tile, V tile) stage, with the group's <= 8 query heads as the N dimension of
// mma.sync.m16n8k16 and the page's 16 tokens as M:
//   S^T[16 x 8] = K_tile . Q_g^T,  online softmax over tokens,  O^T[D x 8] += V_tile^T . P^T.
// K fragments come from ldmatrix, V^T fragments from ldmatrix.trans, P^T is turned from
// accumulator layout into B-operand layout by movmatrix. e4m3 tiles are converted to f16 in
// registers (exact); their per-(page, head) scales multiply the scores (K) and the
// probabilities (V).
#pragma once

#include <cuda_bf16.h>

#include "tma_ptx.cuh"

namespace pda {

// Q^T fragments (B operand of S^T = K.Q^T) of the G heads starting at q_rows: column n = gid
// is head gid of the group, zero for gid >= G.
template <int D, bool kFp8>
__device__ __forceinline__ void load_q_fragments(const __nv_bfloat16* q_rows, int G, int gid, int tq,
                                                 uint32_t (&qf)[D / 16][2]) {
  const __nv_bfloat16* qrow = q_rows + gid * D;
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    qf[ks][0] = 0u; qf[ks][1] = 0u;
    if (gid < G) {
      if (!kFp8) {
        qf[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq);
        qf[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq + 8);
      } else {
        // e4m3 K fragments carry d = 16ks+4tq+{0,1} in k-slots {2tq,2tq+1} and
        // d = 16ks+4tq+{2,3} in k-slots {2tq+8,2tq+9}; q follows the same order.
        const uint2 raw = *reinterpret_cast<const uint2*>(qrow + 16 * ks + 4 * tq);
        const float q0 = __uint_as_float(raw.x << 16), q1 = __uint_as_float(raw.x & 0xffff0000u);
        const float q2 = __uint_as_float(raw.y << 16), q3 = __uint_as_float(raw.y & 0xffff0000u);
        qf[ks][0] = pack2<true>(q0, q1);
        qf[ks][1] = pack2<true>(q2, q3);
      }
    }
  }
}

// One page tile. kt / vt: shared-memory addresses of the landed K and V tiles (128-byte
// swizzled lines); rows [n_skip, n_valid) of the tile are attended; sc = scale * log2(e)
// (* k_scale for e4m3), vsc = v_scale (1 for bf16). (m, l) are this thread's running maxima and
// partial sums for heads 2tq and 2tq+1; o is the O^T accumulator fragment. Warp-collective.
template <int D, bool kFp8>
__device__ __forceinline__ void decode_tile(uint32_t kt, uint32_t vt, int n_valid, int n_skip, float sc,
                                            float vsc, const uint32_t (&qf)[D / 16][2], float& m0,
                                            float& m1, float& l0, float& l1, float (&o)[D / 16][4],
                                            int lane) {
  constexpr int kKSteps = D / 16;
  constexpr int kRowBytes = D * (kFp8 ? 1 : 2);
  constexpr int kPageSize = 16;
  const int gid = lane >> 2;
  // ldmatrix lane addressing: matrix j = lane/8, row-in-matrix = lane%8
  const int lj = lane >> 3, lr = lane & 7;
  const int k_row = lr + 8 * (lj & 1), k_chk = lj >> 1;        // K (and e4m3 V): rows by j&1, chunk by j>>1
  const int v_row = kFp8 ? k_row : lr + 8 * (lj >> 1);         // bf16 V^T: rows by j>>1, chunk by j&1
  const int v_chk = kFp8 ? k_chk : (lj & 1);

    if (n_valid < kPageSize || n_skip > 0) {
      // rows outside the attended range may hold anything: clear them in V (K is masked by select)
      const int n_chunks = kRowBytes / 16;
      const int n_clear = kPageSize - n_valid + n_skip;
      for (int i = lane; i < n_clear * n_chunks; i += 32) {
        int r = i / n_chunks;
        const int ch = i % n_chunks;
        r = r < n_skip ? r : n_valid + (r - n_skip);
        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(vt + tile_off(r, ch)), "r"(0));
      }
      __syncwarp();
    }

    // ---- S^T = K . Q^T
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
    if (!kFp8) {
#pragma unroll
      for (int ks = 0; ks < kKSteps; ++ks) {
        uint32_t a[4];
        ldsm_x4(kt + tile_off(k_row, 2 * ks + k_chk), a);
        if (ks & 1) mma16816<false>(sb, a, qf[ks][0], qf[ks][1]);
        else mma16816<false>(sa, a, qf[ks][0], qf[ks][1]);
      }
    } else {
#pragma unroll
      for (int ks = 0; ks < kKSteps; ks += 2) {
        uint32_t r[4], a[4];
        ldsm_x4(kt + tile_off(k_row, ks + k_chk), r);   // r0,r1: chunk ks rows 0-7 / 8-15; r2,r3: chunk ks+1
        e4m3x4_to_f16x2x2(r[0], a[0], a[2]);
        e4m3x4_to_f16x2x2(r[1], a[1], a[3]);
        mma16816<true>(sa, a, qf[ks][0], qf[ks][1]);
        e4m3x4_to_f16x2x2(r[2], a[0], a[2]);
        e4m3x4_to_f16x2x2(r[3], a[1], a[3]);
        mma16816<true>(sb, a, qf[ks + 1][0], qf[ks + 1][1]);
      }
    }
    float s0 = (sa[0] + sb[0]) * sc, s1 = (sa[1] + sb[1]) * sc;   // token gid,   heads 2tq, 2tq+1
    float s2 = (sa[2] + sb[2]) * sc, s3 = (sa[3] + sb[3]) * sc;   // token gid+8
    if (n_valid < kPageSize || n_skip > 0) {
      if (gid >= n_valid || gid < n_skip) { s0 = -INFINITY; s1 = -INFINITY; }
      if (gid + 8 >= n_valid || gid + 8 < n_skip) { s2 = -INFINITY; s3 = -INFINITY; }
    }

    // ---- online softmax (base 2), max over the tile's tokens = over gid and the two rows
    float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: every tile has an attended row
    const float al0 = ex2(m0 - mn0), al1 = ex2(m1 - mn1);     // ex2(-inf) = 0 on the first tile
    m0 = mn0; m1 = mn1;
    const float p0 = ex2(s0 - mn0), p1 = ex2(s1 - mn1), p2 = ex2(s2 - mn0), p3 = ex2(s3 - mn1);
    l0 = fmaf(l0, al0, p0 + p2);
    l1 = fmaf(l1, al1, p1 + p3);
    const uint32_t pb0 = movmatrix_trans(pack2<kFp8>(p0 * vsc, p1 * vsc));   // P^T rows: tokens 0-7
    const uint32_t pb1 = movmatrix_trans(pack2<kFp8>(p2 * vsc, p3 * vsc));   // tokens 8-15

    // ---- O^T = O^T * alpha + V^T . P^T
    // (after the first tiles of a unit the running maxima seldom move: alpha is exactly 1 then, and the
    // 4 D / 16 multiplications are skipped when it is for the whole warp)
    if (__any_sync(0xffffffffu, (al0 != 1.f) | (al1 != 1.f))) {
#pragma unroll
      for (int mt = 0; mt < kKSteps; ++mt) {
        o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1;
      }
    }
    if (!kFp8) {
#pragma unroll
      for (int mt = 0; mt < kKSteps; ++mt) {
        uint32_t a[4];
        ldsm_x4_trans(vt + tile_off(v_row, 2 * mt + v_chk), a);
        mma16816<false>(o[mt], a, pb0, pb1);
      }
    } else {
#pragma unroll
      for (int mt = 0; mt < kKSteps; mt += 2) {
        uint32_t r[4], a[4];
        ldsm_x4_trans(vt + tile_off(v_row, mt + v_chk), r);
        // a transposed register holds bytes V[2tq][dA], V[2tq][dA+1], V[2tq+1][dA], V[2tq+1][dA+1]
        // with dA = 16*chunk + 2gid: regroup to (V[2tq][d], V[2tq+1][d]) pairs for d = dA, dA+1
#pragma unroll
        for (int i = 0; i < 4; ++i) r[i] = __byte_perm(r[i], 0, 0x3120);
        e4m3x4_to_f16x2x2(r[0], a[0], a[1]);
        e4m3x4_to_f16x2x2(r[1], a[2], a[3]);
        mma16816<true>(o[mt], a, pb0, pb1);
        e4m3x4_to_f16x2x2(r[2], a[0], a[1]);
        e4m3x4_to_f16x2x2(r[3], a[2], a[3]);
        mma16816<true>(o[mt + 1], a, pb0, pb1);
      }
    }

}

}  // namespace pda
