// Softmax / correction / epilogue role of the tcgen05 attention kernel (included by ippd_attn_tc.cuh).
//
// Four warpgroups of 128 threads (warps 2..17).  Thread (wg, row) owns TMEM lane `row` and the 32 S columns
// [32*wg, 32*wg+32) of every key tile: it loads them into registers, takes the maximum over the columns its query row
// may see, exchanges it with the three other owners of the row through shared memory (rounded up to bf16 so that all
// four derive the identical reference maximum), writes its 16 packed words of the P row (bf16) over the S buffer in
// TMEM and keeps a partial row sum.  Rescaling of the O row, Q~ staging and the epilogue are split by output columns
// [wg*D/4, (wg+1)*D/4).  Four warps per SM sub-partition hide each other's TMEM, MUFU and barrier latencies.
#pragma once

#define IPPD_TC_NWG 4  // softmax warpgroups
#define IPPD_TC_CW 32  // S columns per thread

// exp2(s*scale - m) for 8 consecutive S values -> 4 packed bf16 pairs; the sum goes to two accumulators (ILP).
__device__ __forceinline__ void tc_exp8(const uint32_t* s, float scale, float m, uint32_t* p, float& acc0, float& acc1) {
  float e0 = fast_exp2(fmaf(__uint_as_float(s[0]), scale, -m));
  float e1 = fast_exp2(fmaf(__uint_as_float(s[1]), scale, -m));
  float e2 = fast_exp2(fmaf(__uint_as_float(s[2]), scale, -m));
  float e3 = fast_exp2(fmaf(__uint_as_float(s[3]), scale, -m));
  float e4 = fast_exp2(fmaf(__uint_as_float(s[4]), scale, -m));
  float e5 = fast_exp2(fmaf(__uint_as_float(s[5]), scale, -m));
  float e6 = fast_exp2(fmaf(__uint_as_float(s[6]), scale, -m));
  float e7 = fast_exp2(fmaf(__uint_as_float(s[7]), scale, -m));
  p[0] = pack_bf16(e0, e1);
  p[1] = pack_bf16(e2, e3);
  p[2] = pack_bf16(e4, e5);
  p[3] = pack_bf16(e6, e7);
  // the row sum is taken over the ROUNDED probabilities, the ones the P V product really uses, so that the
  // rounding of a dominant key cancels between numerator and denominator
  acc0 += (__uint_as_float(p[0] << 16) + __uint_as_float(p[0] & 0xFFFF0000u)) +
          (__uint_as_float(p[1] << 16) + __uint_as_float(p[1] & 0xFFFF0000u));
  acc1 += (__uint_as_float(p[2] << 16) + __uint_as_float(p[2] & 0xFFFF0000u)) +
          (__uint_as_float(p[3] << 16) + __uint_as_float(p[3] & 0xFFFF0000u));
}

// The 8-bit cache variant: the probabilities enter the P V product as two e4m3 rows, P = P_hi + P_lo (P_hi the
// nearest e4m3 number, P_lo the nearest to the rest), which keeps about 8 significant bits; the exponent is biased so
// that the row's largest probability lies in [2^(BIAS), 2^(BIAS + THRESHOLD)] = [16, 256] and the smallest one that
// survives (2^-9, the e4m3 subnormal step) is 2^-13 of it or less.  The bias multiplies numerator and row sum alike.
#define IPPD_TC8_BIAS 4.0f
#define IPPD_TC8_RESCALE_THRESHOLD 4.0f
// exp2(s*scale - m) for 8 consecutive S values -> 2 words of P_hi and 2 of P_lo (four e4m3 values each, the first in
// the lowest byte); the row sum is taken over the unrounded values.
__device__ __forceinline__ void tc_exp8_f8(const uint32_t* s, float scale, float m, uint32_t* p_hi, uint32_t* p_lo,
                                           float& acc0, float& acc1) {
  uint32_t h16[4], l16[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float e0 = fast_exp2(fmaf(__uint_as_float(s[2 * i]), scale, -m));
    const float e1 = fast_exp2(fmaf(__uint_as_float(s[2 * i + 1]), scale, -m));
    if (i & 1) acc1 += e0 + e1; else acc0 += e0 + e1;
    const __half2 e = __floats2half2_rn(e0, e1);
    const __nv_fp8x2_storage_t hi = __nv_cvt_halfraw2_to_fp8x2(static_cast<__half2_raw>(e), __NV_SATFINITE, __NV_E4M3);
    const __half2 back = __half2(__nv_cvt_fp8x2_to_halfraw2(hi, __NV_E4M3));
    const __half2 rest = __hsub2(e, back);  // exact: the two are within a factor of two of each other
    const __nv_fp8x2_storage_t lo = __nv_cvt_halfraw2_to_fp8x2(static_cast<__half2_raw>(rest), __NV_SATFINITE, __NV_E4M3);
    h16[i] = hi;
    l16[i] = lo;
  }
  p_hi[0] = h16[0] | (h16[1] << 16);
  p_hi[1] = h16[2] | (h16[3] << 16);
  p_lo[0] = l16[0] | (l16[1] << 16);
  p_lo[1] = l16[2] | (l16[3] << 16);
}
// Four floats -> the e4m3 numbers nearest to them (a word) and nearest to what is left (another word).
__device__ __forceinline__ void tc_split_e4m3x4(float a, float b, float c, float d, uint32_t& hi, uint32_t& lo) {
  const __nv_fp8x2_storage_t h0 = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
  const __nv_fp8x2_storage_t h1 = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
  const float2 b0 = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2(h0, __NV_E4M3)));
  const float2 b1 = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2(h1, __NV_E4M3)));
  const __nv_fp8x2_storage_t l0 = __nv_cvt_float2_to_fp8x2(make_float2(a - b0.x, b - b0.y), __NV_SATFINITE, __NV_E4M3);
  const __nv_fp8x2_storage_t l1 = __nv_cvt_float2_to_fp8x2(make_float2(c - b1.x, d - b1.y), __NV_SATFINITE, __NV_E4M3);
  hi = (uint32_t)h0 | ((uint32_t)h1 << 16);
  lo = (uint32_t)l0 | ((uint32_t)l1 << 16);
}

// Upper 16 bits of the smallest bf16 value >= x: the exchanged maximum must not be smaller than the true one, so that
// every probability stays <= 1.  (Positive: round the magnitude up; negative: truncate it.)
__device__ __forceinline__ unsigned short tc_bf16_ceil_bits(float x) {
  const uint32_t b = __float_as_uint(x);
  return (unsigned short)(((b & 0x80000000u) ? b : b + 0xFFFFu) >> 16);
}

// Barrier of the four warps (one per warpgroup) that own the same 32 TMEM lanes: hardware named barriers 2..5.
// A named barrier cannot time out, so its passes follow a fixed schedule that depends only on the CTA's segment list
// (one pass per tile, three per segment epilogue): a warp that gives up (a bounded wait ran out, or another role raised
// the abort flag) still makes the passes it owes (see the end of tc_softmax_role), so nobody is left waiting.
// All lanes of a warp execute every wait converged on one barrier and so see the same outcome.
__device__ __forceinline__ void tc_quad_sync(int warp) {
  asm volatile("bar.sync %0, 128;" ::"r"(2 + (warp & 3)) : "memory");
}
// A softmax warp that gives up makes the passes it still owes: `owed_here` in its current segment, plus one per tile
// and three per epilogue for every later segment of the CTA's slice [g, g1) (g = first tile after the current segment;
// the walk repeats tc_next_segment's cuts).  Kept out of line: it must not cost the hot loop registers.
__device__ __noinline__ void tc_quad_give_up(const int32_t* rb_tile_begin, int n_rb, int T1, long long g, long long g1,
                                             int owed_here, int warp) {
  long long owed = owed_here;
  while (g < g1) {
    const int within = (int)(g % T1);
    int rb = 0;
    while (rb + 1 < n_rb && rb_tile_begin[rb + 1] <= within) ++rb;
    const long long end = min((long long)rb_tile_begin[rb + 1], (long long)within + (g1 - g));
    owed += (end - within) + 3;
    g += end - within;
  }
  for (long long k = 0; k < owed; ++k) tc_quad_sync(warp);
}

template <int D, class SH = TcShared, bool KV8 = false>
__device__ __forceinline__ void tc_softmax_role(const IppdDev& L, const IppdStepDev& S, const IppdTcArgs& A,
                                                SH* sh, uint32_t tmem, long long g0, long long g1,
                                                const __nv_bfloat16* __restrict__ q_raw, void* __restrict__ out,
                                                float* __restrict__ part_o, float* __restrict__ part_ml) {
  constexpr int DQ = D / IPPD_TC_NWG;  // output columns per warpgroup (32 or 16)
  constexpr int NW = D / 16;           // packed Q~ words (bf16 pairs) per warpgroup and rotation half (8 or 4)
  constexpr unsigned FULL = 0xffffffffu;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wg = (warp - 2) >> 2;          // 0..3
  const int row = (warp & 3) * 32 + lane;  // TMEM lane this thread may access = query row
  const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
  const uint32_t tS0 = tmem, tO = tmem + 256, tQ = tmem + 384;
  const int Hkv = L.Hkv, G = L.G;
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
  const int my_q = row / G;  // question (local to the row block) of my row

  // Stages this warpgroup's part of Q~ of segment `sq` into TMEM buffer `qbuf` (the A operand of S = Q~ K^T: lane = row,
  // column c holds the bf16 pair (2c, 2c+1) of the row) and signals the MMA warp.  The buffer was last read by the S
  // MMAs of the segment before the previous one, which are long complete.
  // 8-bit cache variant: the row is scaled by a power of two that brings its largest magnitude to [64, 182) (from the
  // largest raw magnitude: the rotation grows a value by less than sqrt 2), split into Q~_hi + Q~_lo (two e4m3 rows,
  // four values per column; hi at columns [0, D/4), lo at [D/4, D/2)), and the inverse factor goes into the score
  // scale of the row, which the call returns.
  auto stage_q8 = [&](const TcSegment& sq, uint32_t qbuf) -> float {
    constexpr int NV = D / 8;  // values per warpgroup and rotation half (16 or 8)
    const IppdRowBlock rb = S.rbs[sq.rb];
    const int nrows = rb.n_act * G;
    uint32_t hl[NV / 4], hh[NV / 4], ll_[NV / 4], lh[NV / 4];
    float inv_f = 1.f;
    if (row < nrows) {
      const int j = row - my_q * G, ai = rb.act_begin + my_q;
      const int pos = S.act_pos[ai];
      const __nv_bfloat16* qp = q_raw + (((size_t)sq.ll * S.A + ai) * L.Hq + sq.head * G + j) * D;
      uint32_t mx = 0;  // largest magnitude of the raw row, as bf16 bits (they order like integers)
#pragma unroll
      for (int c = 0; c < D / 8; ++c) {
        const uint4 w = *reinterpret_cast<const uint4*>(qp + c * 8);
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) mx = max(mx, max(ws[e] & 0x7FFFu, (ws[e] >> 16) & 0x7FFFu));
      }
      int field = 260 - (int)(mx >> 7);  // exponent field of 2^(6 - floor(log2 max))
      field = min(250, max(4, field));
      const float f = __uint_as_float((uint32_t)field << 23);
      inv_f = __uint_as_float((uint32_t)(254 - field) << 23);
      const float2* cs = L.rope + (size_t)pos * (D / 2);
      float ql[NV], qh[NV];
#pragma unroll
      for (int cc = 0; cc < NV / 8; ++cc) {
        const int c = wg * (NV / 8) + cc;  // 16-byte chunk c of the raw row and its rotation partner c + D/16
        uint4 lo = *reinterpret_cast<const uint4*>(qp + c * 8);
        uint4 hi = *reinterpret_cast<const uint4*>(qp + c * 8 + D / 2);
        const __nv_bfloat162* pl = reinterpret_cast<const __nv_bfloat162*>(&lo);
        const __nv_bfloat162* ph = reinterpret_cast<const __nv_bfloat162*>(&hi);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 c0 = cs[c * 8 + 2 * e], c1 = cs[c * 8 + 2 * e + 1];
          float l0 = __bfloat162float(pl[e].x) * f, l1 = __bfloat162float(pl[e].y) * f;
          float h0 = __bfloat162float(ph[e].x) * f, h1 = __bfloat162float(ph[e].y) * f;
          ql[cc * 8 + 2 * e] = l0 * c0.x - h0 * c0.y;
          ql[cc * 8 + 2 * e + 1] = l1 * c1.x - h1 * c1.y;
          qh[cc * 8 + 2 * e] = h0 * c0.x + l0 * c0.y;
          qh[cc * 8 + 2 * e + 1] = h1 * c1.x + l1 * c1.y;
        }
      }
#pragma unroll
      for (int e = 0; e < NV / 4; ++e) {
        tc_split_e4m3x4(ql[4 * e], ql[4 * e + 1], ql[4 * e + 2], ql[4 * e + 3], hl[e], ll_[e]);
        tc_split_e4m3x4(qh[4 * e], qh[4 * e + 1], qh[4 * e + 2], qh[4 * e + 3], hh[e], lh[e]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < NV / 4; ++e) { hl[e] = 0u; hh[e] = 0u; ll_[e] = 0u; lh[e] = 0u; }
    }
    // values d = (NV wg ..) sit in columns NV/4 * wg .., their rotation partners D/8 columns further; lo rows D/4 further
    const uint32_t tq = tQ + qbuf * 64 + lane_base + wg * (NV / 4);
    if constexpr (NV == 16) {
      { uint32_t* w = hl; TC_ST4(tq, w); }
      { uint32_t* w = hh; TC_ST4(tq + D / 8, w); }
      { uint32_t* w = ll_; TC_ST4(tq + D / 4, w); }
      { uint32_t* w = lh; TC_ST4(tq + D / 4 + D / 8, w); }
    } else {
      { uint32_t* w = hl; TC_ST2(tq, w); }
      { uint32_t* w = hh; TC_ST2(tq + D / 8, w); }
      { uint32_t* w = ll_; TC_ST2(tq + D / 4, w); }
      { uint32_t* w = lh; TC_ST2(tq + D / 4 + D / 8, w); }
    }
    tc_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh->q_full);
    return scale_log2 * inv_f;
  };
  float sc_cur = scale_log2, sc_next = scale_log2;  // score scale of my row (8-bit variant: with the row's factor)
  (void)sc_next;
  auto stage_q = [&](const TcSegment& sq, uint32_t qbuf) {
    if constexpr (KV8) {
      sc_next = stage_q8(sq, qbuf);
      return;
    }
    const IppdRowBlock rb = S.rbs[sq.rb];
    const int nrows = rb.n_act * G;
    uint32_t wlo[NW], whi[NW];  // rotated pairs d in [2*NW*wg, 2*NW*(wg+1)) and the same + D/2
    if (row < nrows) {
      const int j = row - my_q * G, ai = rb.act_begin + my_q;
      const int pos = S.act_pos[ai];
      const __nv_bfloat16* qp = q_raw + (((size_t)sq.ll * S.A + ai) * L.Hq + sq.head * G + j) * D;
      const float2* cs = L.rope + (size_t)pos * (D / 2);
#pragma unroll
      for (int cc = 0; cc < NW / 4; ++cc) {
        const int c = wg * (NW / 4) + cc;  // 16-byte chunk c and its rotation partner c + D/16
        uint4 lo = *reinterpret_cast<const uint4*>(qp + c * 8);
        uint4 hi = *reinterpret_cast<const uint4*>(qp + c * 8 + D / 2);
        const __nv_bfloat162* pl = reinterpret_cast<const __nv_bfloat162*>(&lo);
        const __nv_bfloat162* ph = reinterpret_cast<const __nv_bfloat162*>(&hi);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float2 c0 = cs[c * 8 + 2 * e], c1 = cs[c * 8 + 2 * e + 1];
          float l0 = __bfloat162float(pl[e].x), l1 = __bfloat162float(pl[e].y);
          float h0 = __bfloat162float(ph[e].x), h1 = __bfloat162float(ph[e].y);
          wlo[cc * 4 + e] = pack_bf16(l0 * c0.x - h0 * c0.y, l1 * c1.x - h1 * c1.y);
          whi[cc * 4 + e] = pack_bf16(h0 * c0.x + l0 * c0.y, h1 * c1.x + l1 * c1.y);
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < NW; ++e) { wlo[e] = 0u; whi[e] = 0u; }
    }
    const uint32_t tq = tQ + qbuf * 64 + lane_base + wg * NW;
    if constexpr (NW == 8) {
      { uint32_t* w = wlo; TC_ST8(tq, w); }
      { uint32_t* w = whi; TC_ST8(tq + D / 4, w); }
    } else {
      { uint32_t* w = wlo; TC_ST4(tq, w); }
      { uint32_t* w = whi; TC_ST4(tq + D / 4, w); }
    }
    tc_wait_st();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh->q_full);
  };

  int gofs = 0;  // position in the CTA's slice, relative to g0 (a 32-bit value: this role is short of registers)
  TcSegment sg;
  uint32_t jt = 0, nseg = 0;
  bool have;
  {
    long long g = g0;
    have = tc_next_segment(A, S, Hkv, g0, g1, g, sg);
    gofs = (int)(g - g0);
  }
  if (have) stage_q(sg, 0);
  while (have) {
    if constexpr (KV8) sc_cur = sc_next;  // staged with this segment's Q~ (before the loop or during the last segment)
    const float sc = KV8 ? sc_cur : scale_log2;
    const IppdRowBlock rb = S.rbs[sg.rb];
    const int nrows = rb.n_act * G;
    // A context tile is seen whole by every query row, so a warp with at least one query row takes the path without
    // per-lane windows and votes for it; its lanes beyond the row block's rows carry a zero Q~ row (S = 0 there), run
    // along and are never stored.  (Taking the windowed path whenever a warp was only partly filled made a context
    // tile 1.5x slower for every row block whose row count is not a multiple of 32.)
    const bool warp_has_rows = __any_sync(FULL, row < nrows);

    float m_ref = -INFINITY, l_sum = 0.f;  // l_sum: this thread's part of the row sum
    const int nt = sg.t_end - sg.t_begin;
    for (int i = 0; i < nt; ++i, ++jt) {
      if (!tc_wait(&sh->s_full[jt & 1], (jt >> 1) & 1, L, sh)) { tc_quad_give_up(A.rb_tile_begin, S.n_rb, A.T1, g0 + gofs, g1, nt - i + 3, warp); return; }
      tc_fence_after();
      // the tile's description was staged by the producer before its K copy, which S(jt) has consumed
      const TcMeta& meta = sh->meta[jt % SH::kNMeta];
      const int tile_rows = meta.rows, n_pieces = meta.n_pieces;
      const int base = wg * IPPD_TC_CW;              // my first column
      const bool part_used = tile_rows > base;       // the P V product reads my columns of the P row
      int lo, hi, wlo, whi;
      bool mine, warp_any, all_full;
      if (n_pieces == 0 && warp_has_rows) {
        // context tile: no per-lane window, no votes
        lo = 0;
        hi = min(IPPD_TC_CW, max(0, tile_rows - base));
        mine = warp_any = hi > 0;
        all_full = hi == IPPD_TC_CW;
        wlo = 0;
        whi = (hi + 7) & ~7;
      } else {
        // columns [c0, c1) of the tile my query row may see, cut to my 32 columns
        int c0 = 0, c1 = 0;
        if (row < nrows) {
          if (n_pieces == 0) {
            c1 = tile_rows;
          } else {
            // the producer has reduced the tile's pieces to one column window per question
            c0 = meta.c0[my_q];
            c1 = meta.c1[my_q];
          }
        }
        lo = min(IPPD_TC_CW, max(0, c0 - base));
        hi = min(IPPD_TC_CW, max(0, c1 - base));
        mine = hi > lo;
        warp_any = __any_sync(FULL, mine);
        all_full = __all_sync(FULL, lo == 0 && hi == IPPD_TC_CW);
        wlo = __reduce_min_sync(FULL, mine ? lo : IPPD_TC_CW) & ~7;  // 8-aligned union of the warp's windows
        whi = (__reduce_max_sync(FULL, mine ? hi : 0) + 7) & ~7;
      }
      const uint32_t tS = tS0 + (jt & 1) * 128 + base + lane_base;
      const uint32_t tP = tS0 + (jt & 1) * 128 + wg * (IPPD_TC_CW / 2) + lane_base;  // P overwrites the head of S
      uint32_t s[IPPD_TC_CW];
      // ---- maximum over my window (raw scores; the scale is positive), four independent chains ----
      float mloc = -INFINITY;
      if (warp_any) {
        TC_LD32(tS, s);
        tc_wait_ld();
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
        if (all_full) {
#pragma unroll
          for (int e = 0; e < IPPD_TC_CW; e += 4) {
            m0 = fmaxf(m0, __uint_as_float(s[e]));
            m1 = fmaxf(m1, __uint_as_float(s[e + 1]));
            m2 = fmaxf(m2, __uint_as_float(s[e + 2]));
            m3 = fmaxf(m3, __uint_as_float(s[e + 3]));
          }
        } else {
          // entries outside [lo, hi) are masked (another question's piece, or beyond the valid tokens)
#pragma unroll
          for (int e = 0; e < IPPD_TC_CW; e += 4) {
            if (e >= wlo && e < whi) {
              float v0 = (e >= lo && e < hi) ? __uint_as_float(s[e]) : -INFINITY;
              float v1 = (e + 1 >= lo && e + 1 < hi) ? __uint_as_float(s[e + 1]) : -INFINITY;
              float v2 = (e + 2 >= lo && e + 2 < hi) ? __uint_as_float(s[e + 2]) : -INFINITY;
              float v3 = (e + 3 >= lo && e + 3 < hi) ? __uint_as_float(s[e + 3]) : -INFINITY;
              s[e] = __float_as_uint(v0);
              s[e + 1] = __float_as_uint(v1);
              s[e + 2] = __float_as_uint(v2);
              s[e + 3] = __float_as_uint(v3);
              m0 = fmaxf(m0, v0); m1 = fmaxf(m1, v1); m2 = fmaxf(m2, v2); m3 = fmaxf(m3, v3);
            }
          }
        }
        mloc = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * sc;
      }
      // exchange the quarter-row maxima, rounded up to bf16 so that all four owners derive the same reference; the
      // barrier also orders every owner's S loads before the P stores below, which overwrite S columns of other owners
      const unsigned short mbits = tc_bf16_ceil_bits(mloc);
      sh->xmax[jt & 1][wg][row] = mbits;
      tc_quad_sync(warp);
      float mt;
      {
        const unsigned short b0 = sh->xmax[jt & 1][0][row], b1 = sh->xmax[jt & 1][1][row];
        const unsigned short b2 = sh->xmax[jt & 1][2][row], b3 = sh->xmax[jt & 1][3][row];
        mt = fmaxf(fmaxf(__uint_as_float((uint32_t)b0 << 16), __uint_as_float((uint32_t)b1 << 16)),
                   fmaxf(__uint_as_float((uint32_t)b2 << 16), __uint_as_float((uint32_t)b3 << 16)));
      }
      // lazy rescale: keep the old reference unless the row's maximum grew past the threshold (or it is the first)
      const bool grow = mt > m_ref + (KV8 ? IPPD_TC8_RESCALE_THRESHOLD : IPPD_TC_RESCALE_THRESHOLD) ||
                        (m_ref == -INFINITY && mt > -INFINITY);
      float alpha = 1.f;
      if (grow) {
        alpha = fast_exp2(m_ref - mt);  // 0 when this is the row's first visible tile
        m_ref = mt;
        l_sum *= alpha;
      }
      if (i > 0 && __any_sync(FULL, grow)) {
        // rare: rescale my quarter of the O row, which needs PV(jt-1) to have finished
        if (!tc_wait(&sh->pv_done[(jt - 1) & 1], ((jt - 1) >> 1) & 1, L, sh)) { tc_quad_give_up(A.rb_tile_begin, S.n_rb, A.T1, g0 + gofs, g1, nt - i - 1 + 3, warp); return; }
        tc_fence_after();
        uint32_t o[DQ];
        if constexpr (DQ == 32) { TC_LD32(tO + lane_base + wg * DQ, o); } else { TC_LD16(tO + lane_base + wg * DQ, o); }
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < DQ; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
        if constexpr (DQ == 32) { TC_ST32(tO + lane_base + wg * DQ, o); } else { TC_ST16(tO + lane_base + wg * DQ, o); }
      }
      // ---- my 16 packed words of the P row (zeros where my row sees nothing) ----
      if (part_used) {
        uint32_t p[IPPD_TC_CW / 2];
        if constexpr (KV8) {
          // p[0..7]: my 32 tokens of P_hi (columns 8 wg .. of the S buffer), p[8..15]: of P_lo (32 columns further)
          if (warp_any) {
            const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref - IPPD_TC8_BIAS;
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int e = 0; e < IPPD_TC_CW; e += 8) {
              if (e >= wlo && e < whi) tc_exp8_f8(s + e, sc, m_use, p + e / 4, p + 8 + e / 4, a0, a1);
              else { p[e / 4] = 0u; p[e / 4 + 1] = 0u; p[8 + e / 4] = 0u; p[8 + e / 4 + 1] = 0u; }
            }
            l_sum += a0 + a1;
          } else {
#pragma unroll
            for (int e = 0; e < IPPD_TC_CW / 2; ++e) p[e] = 0u;
          }
          const uint32_t tP8 = tS0 + (jt & 1) * 128 + wg * (IPPD_TC_CW / 4) + lane_base;
          { uint32_t* w = p; TC_ST8(tP8, w); }
          { uint32_t* w = p + 8; TC_ST8(tP8 + 32, w); }
        } else {
        if (warp_any) {
          const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;  // rows that see nothing yet: exp2(-inf) = 0
          float a0 = 0.f, a1 = 0.f;
#pragma unroll
          for (int e = 0; e < IPPD_TC_CW; e += 8) {
            if (e >= wlo && e < whi) tc_exp8(s + e, scale_log2, m_use, p + e / 2, a0, a1);
            else { p[e / 2] = 0u; p[e / 2 + 1] = 0u; p[e / 2 + 2] = 0u; p[e / 2 + 3] = 0u; }
          }
          l_sum += a0 + a1;
        } else {
#pragma unroll
          for (int e = 0; e < IPPD_TC_CW / 2; ++e) p[e] = 0u;
        }
        TC_ST16(tP, p);
        }
      }
      tc_wait_st();  // the P words and a possible O rescale
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->p_full[jt & 1]);
    }
    // ---- the next segment's Q~ goes to the other TMEM buffer now, so that the MMA warp can start its first S tiles
    // while this segment's epilogue runs ----
    TcSegment nx;
    long long g_next = g0 + gofs;
    const bool have_next = tc_next_segment(A, S, Hkv, g0, g1, g_next, nx);
    if (have_next) stage_q(nx, (nseg + 1) & 1);
    // ---- epilogue: total row sum (exchanged through my row's own maxima slots: low half in parity 0, high half in
    // parity 1), wait for the last PV, store my quarter of the O row ----
    tc_quad_sync(warp);  // my row's other owners have read the last tile's maxima
    {
      const uint32_t lb = __float_as_uint(l_sum);
      sh->xmax[0][wg][row] = (unsigned short)(lb & 0xFFFFu);
      sh->xmax[1][wg][row] = (unsigned short)(lb >> 16);
    }
    tc_quad_sync(warp);
    float l_tot = 0.f;
#pragma unroll
    for (int w = 0; w < IPPD_TC_NWG; ++w)
      l_tot += __uint_as_float((uint32_t)sh->xmax[0][w][row] | ((uint32_t)sh->xmax[1][w][row] << 16));
    tc_quad_sync(warp);  // the slots go back to the maxima of the next tiles
    if (!tc_wait(&sh->pv_done[(jt - 1) & 1], ((jt - 1) >> 1) & 1, L, sh)) { tc_quad_give_up(A.rb_tile_begin, S.n_rb, A.T1, g0 + gofs, g1, 0, warp); return; }
    tc_fence_after();
    {
      const bool valid_row = row < nrows;
      const int a = valid_row ? my_q : 0, j = row - a * G;
      const float inv = (sg.complete && l_tot > 0.f) ? 1.f / l_tot : 1.f;
      size_t obase = (((size_t)sg.ll * S.A + rb.act_begin + a) * L.Hq + sg.head * G + j) * D + wg * DQ;
      size_t pslot = (size_t)blockIdx.x * 2 + sg.slot;
      float* po = part_o + (pslot * IPPD_TC_ROWS + row) * D + wg * DQ;
      uint32_t o[DQ];
      if constexpr (DQ == 32) { TC_LD32(tO + lane_base + wg * DQ, o); } else { TC_LD16(tO + lane_base + wg * DQ, o); }
      tc_wait_ld();
      if (valid_row) {
        if (sg.complete) {
          if (A.out_f32) {
            float* dst = reinterpret_cast<float*>(out) + obase;
#pragma unroll
            for (int e = 0; e < DQ; e += 4)
              *reinterpret_cast<float4*>(dst + e) =
                  make_float4(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv,
                              __uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + obase;
#pragma unroll
            for (int e = 0; e < DQ; e += 8) {
              uint4 pk;
              pk.x = pack_bf16(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
              pk.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
              pk.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
              pk.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
              *reinterpret_cast<uint4*>(dst + e) = pk;
            }
          }
        } else {
#pragma unroll
          for (int e = 0; e < DQ; e += 4)
            *reinterpret_cast<float4*>(po + e) = make_float4(__uint_as_float(o[e]), __uint_as_float(o[e + 1]),
                                                             __uint_as_float(o[e + 2]), __uint_as_float(o[e + 3]));
        }
      }
      if (valid_row && !sg.complete && wg == 0) {
        float* pm = part_ml + (pslot * IPPD_TC_ROWS + row) * 2;
        pm[0] = m_ref;
        pm[1] = l_tot;
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sh->o_free);
    ++nseg;
    sg = nx;
    gofs = (int)(g_next - g0);
    have = have_next;
  }
}
