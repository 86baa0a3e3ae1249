// The per-warp, per-key-tile body of Algorithm 1 (its mixed-precision sections):
// low-precision logits, threats and visiting order, stage 1 (eq. (7)), exponentials,
// lambda / omega update, stage 2 (eq. (8)) and the stage-2 recomputation.
//
// Lane layout.  A warp owns 32 query rows (one group).  Lane l = 4*a + theta holds,
// for the query quad 4a..4a+3 and the 16 keys of sub-block theta, the 64 logits of
// the first pass.  The per-row state (mu, omega) of a quad is replicated in its four
// theta lanes, which all compute it identically.  A 16-bit recomputation of one
// sub-block is shared by the whole warp: lane (a, t) takes the quad's 4 queries and
// keys 4t..4t+3 of that sub-block.
#pragma once
#include "lamp_common.cuh"

namespace lamp {

struct TileGeom {
  int i0;       // first key of the tile
  int j0;       // first query row of the group
  int causal, window;
  bool full;    // every pair of (group x tile) is visible
};

template <bool FULL>
__device__ __forceinline__ bool vis(const TileGeom& g, int i, int j) {
  return FULL || pair_valid(g.causal, g.window, g.i0 + i, g.j0 + j);
}

// First pass: Y8[i][j] = chain over kk of c <- RNE_e4m3(fma(k, q*scale, c)), c0 = +0
// (Alg. 1 "accumulate Y in low precision"; Sec. 4.1 round(c + a*b)).
// qs: this lane's quad inside the transposed, pre-scaled Q tile  [D][qstride]
// kf: this lane's sub-block inside the fp32 K tile               [D][kKfStride]
template <int D>
__device__ __forceinline__ void chain8(const float* __restrict__ qs, int qstride,
                                       const float* __restrict__ kf, float (&acc)[4][16]) {
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 16; ++b) acc[a][b] = 0.0f;
#pragma unroll 2
  for (int kk = 0; kk < D; ++kk) {
    const float4 qv = *reinterpret_cast<const float4*>(qs + kk * qstride);
    const float q4[4] = {qv.x, qv.y, qv.z, qv.w};
    float kv[16];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float4 t = *reinterpret_cast<const float4*>(kf + kk * kKfStride + 4 * c);
      kv[4 * c] = t.x; kv[4 * c + 1] = t.y; kv[4 * c + 2] = t.z; kv[4 * c + 3] = t.w;
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 16; b += 2) {
        float t0 = __fmaf_rn(kv[b], q4[a], acc[a][b]);
        float t1 = __fmaf_rn(kv[b + 1], q4[a], acc[a][b + 1]);
        rne_e4m3_x2(t0, t1);
        acc[a][b] = t0;
        acc[a][b + 1] = t1;
      }
  }
}

// 16-bit logits of sub-block th for this lane's (quad x 4 keys): a sequential fp64
// fma chain over kk, scaled, rounded once to e4m11.
// kf: fp32 K tile base; qrow: global bf16 pointer to the quad's first row.
template <int D>
__device__ __forceinline__ void dot16(const float* __restrict__ kf, const __nv_bfloat16* qrow,
                                      int64_t qstride, int th, int tp, double scale_d,
                                      float (&y)[4][4]) {
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  const float* kcol = kf + kf_pos(16 * th + 4 * tp);
  for (int k0 = 0; k0 < D; k0 += 8) {
    uint4 qraw[4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
      qraw[a] = *reinterpret_cast<const uint4*>(qrow + a * qstride + k0);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float4 kq = *reinterpret_cast<const float4*>(kcol + (k0 + e) * kKfStride);
      const double kd[4] = {(double)kq.x, (double)kq.y, (double)kq.z, (double)kq.w};
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const uint32_t w = (&qraw[a].x)[e >> 1];
        const double qd = (double)__uint_as_float((e & 1) ? (w & 0xffff0000u) : (w << 16));
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fma(kd[b], qd, acc[a][b]);
      }
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) y[a][b] = rne_e4m11(__dmul_rn(scale_d, acc[a][b]));
}

// active, s1, s2, hist, bigrow are warp-uniform; sat8, sat16, gt1 are per-lane partial
// counts that the caller adds up over the warp.
struct WarpCounters {
  unsigned long long active, s1, s2, hist[5], bigrow;
  unsigned int sat8, sat16, gt1;
};

// Row state of a lane's query quad.
struct RowState {
  float mu[4];
  float om[4];
};

// Everything between "accumulate Y in low precision" and the P V product of Alg. 1
// for one (group, key tile).  On return es[key][query] (a [64][32] fp32 tile in
// shared memory, private to the warp) holds the exponentials E_hat, lam[] the
// rescale factors lambda_hat of this lane's quad, st the updated (mu, omega), and the
// flag byte (bits 0-3 stage 1, bits 4-7 stage 2) is returned.
template <int D, bool FULL, bool DUMP>
__device__ __forceinline__ uint32_t lamp_tile(const KernelParams& P, const TileGeom& g,
                                              const float* qs_quad, int qstride,
                                              const float* kf, const __nv_bfloat16* qrow,
                                              const uint32_t* lut, float* es, RowState& st,
                                              float (&lam)[4], WarpCounters& wc,
                                              unsigned long long (&cks)[2], int row_in_dump0) {
  const int lane = threadIdx.x & 31;
  const int qa = lane >> 2, th_own = lane & 3;
  const double scale_d = (double)P.scale;
  const bool force16 = P.flags & LAMP_FORCE_16BIT;
  const bool force8 = P.flags & LAMP_FORCE_8BIT;
  const bool skip1 = (P.flags & (LAMP_FORCE_8BIT | LAMP_NO_STAGE1)) != 0;

  // ---- first pass ---------------------------------------------------------------
  float acc[4][16];
  chain8<D>(qs_quad, qstride, kf + kf_pos(16 * th_own), acc);

  // ---- per sub-block, per query maxima; which sub-blocks are active ----------------
  float cm[4];
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    float m = -INFINITY;
#pragma unroll
    for (int b = 0; b < 16; ++b)
      if (vis<FULL>(g, 16 * th_own + b, 4 * qa + a)) m = fmaxf(m, acc[a][b]);
    cm[a] = m;
  }
  uint32_t actmask = 0;
#pragma unroll
  for (int th = 0; th < 4; ++th) {
    bool act = true;
    if (!FULL) {
      const int s0 = g.i0 + 16 * th;
      act = (!g.causal || s0 <= g.j0 + 31) && (g.window == 0 || g.j0 - (s0 + 15) < g.window);
    }
    actmask |= (uint32_t)act << th;
  }
  const int nact = __popc(actmask);

  // ---- threats T_theta against the maxima at tile start, visiting order --------------
  float tl = -INFINITY;
#pragma unroll
  for (int a = 0; a < 4; ++a)
    if (cm[a] > -INFINITY) tl = fmaxf(tl, __fsub_rn(cm[a], st.mu[a]));
  tl = fmaxf(tl, __shfl_xor_sync(kFull, tl, 4));
  tl = fmaxf(tl, __shfl_xor_sync(kFull, tl, 8));
  tl = fmaxf(tl, __shfl_xor_sync(kFull, tl, 16));
  float T[4];
#pragma unroll
  for (int th = 0; th < 4; ++th) T[th] = __shfl_sync(kFull, tl, th);
  uint32_t order = 0;   // 2 bits per rank: the sub-block visited at that rank
#pragma unroll
  for (int th = 0; th < 4; ++th) {
    int rank = 0;
#pragma unroll
    for (int o = 0; o < 4; ++o)
      if (o != th && ((actmask >> o) & 1u) && (T[o] > T[th] || (T[o] == T[th] && o < th))) ++rank;
    if ((actmask >> th) & 1u) order |= (uint32_t)th << (2 * rank);
  }

  // ---- stage 1: eq. (7), sub-blocks in threat order -----------------------------------
  float muh[4];
#pragma unroll
  for (int a = 0; a < 4; ++a) muh[a] = st.mu[a];
  uint32_t Theta = 0;
  float* es_lane = es + (4 * th_own) * kBQ + 4 * qa;   // [key 16*th + 4*tp + b][query 4*qa + a]
  for (int r = 0; r < nact; ++r) {
    const int th = (order >> (2 * r)) & 3;
    bool fail;
    if (force16) fail = true;
    else if (skip1) fail = false;
    else {
      bool f = false;
      if (th_own == th) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
          if (cm[a] > -INFINITY) {
            const float rhs = __fadd_rn(cm[a], __fmul_rn(fabsf(muh[a]), P.delta));
            if (isinf(muh[a]) || !(muh[a] > rhs)) f = true;
          }
      }
      fail = __any_sync(kFull, f);
    }
    if (!fail) continue;
    Theta |= 1u << th;
    float y[4][4];
    dot16<D>(kf, qrow, P.qs[2], th, th_own, scale_d, y);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      float m = -INFINITY;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        es_lane[(16 * th + b) * kBQ + a] = y[a][b];
        if (vis<FULL>(g, 16 * th + 4 * th_own + b, 4 * qa + a)) {
          m = fmaxf(m, y[a][b]);
          wc.sat16 += fabsf(y[a][b]) == 448.0f;
        }
      }
      m = fmaxf(m, __shfl_xor_sync(kFull, m, 1));
      m = fmaxf(m, __shfl_xor_sync(kFull, m, 2));
      muh[a] = fmaxf(muh[a], m);
    }
  }
  if (skip1 && !force16) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      float m = cm[a];
      m = fmaxf(m, __shfl_xor_sync(kFull, m, 1));
      m = fmaxf(m, __shfl_xor_sync(kFull, m, 2));
      muh[a] = fmaxf(muh[a], m);
    }
  }

  // ---- exponentials: 8-bit through the table, 16-bit correctly rounded ----------------
  const bool own_act = (actmask >> th_own) & 1u;
  const bool own8 = own_act && !((Theta >> th_own) & 1u);
  double rs8[4] = {0.0, 0.0, 0.0, 0.0};
  if (own_act) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const float m8 = trunc_e4m3(muh[a]);
#pragma unroll
      for (int b = 0; b < 16; ++b) {
        const bool ok = vis<FULL>(g, 16 * th_own + b, 4 * qa + a);
        float e = 0.0f;
        if (ok) {
          const float y8 = acc[a][b];
          uint32_t eb = 0xffu;
          wc.sat8 += fabsf(y8) == 448.0f;
          if (own8) {
            const uint32_t w = lut[shift_index(__fsub_rn(m8, y8))];
            e = __uint_as_float(w & 0xffffff00u);
            eb = w & 0xffu;
          }
          if (DUMP) {
            const uint32_t yb = enc_e4m3(y8);
            const uint64_t idx = (uint64_t)((16 * th_own + b) * kBQ + 4 * qa + a) << 8;
            cks[0] += mix64(idx | yb);
            cks[1] += mix64(idx | eb);
            if (row_in_dump0 >= 0) {
              const size_t off = (size_t)(row_in_dump0 + 4 * qa + a) * P.seqlen + g.i0 + 16 * th_own + b;
              if (P.dbg_y8) P.dbg_y8[off] = (uint8_t)yb;
              if (P.dbg_e8) P.dbg_e8[off] = (uint8_t)eb;
            }
          }
        }
        acc[a][b] = e;
        rs8[a] += (double)e;
      }
    }
  } else {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 16; ++b) acc[a][b] = 0.0f;
  }

  double rs16[4] = {0.0, 0.0, 0.0, 0.0};
  auto exp_block = [&](int th) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        float* slot = es_lane + (16 * th + b) * kBQ + a;
        float e = 0.0f;
        if (vis<FULL>(g, 16 * th + 4 * th_own + b, 4 * qa + a)) {
          e = exp16(rne_sig12(__fsub_rn(*slot, muh[a])));
          wc.gt1 += e > 1.0f;
        }
        *slot = e;
        rs16[a] += (double)e;
      }
  };
  for (int th = 0; th < 4; ++th)
    if ((Theta >> th) & 1u) exp_block(th);

  // ---- lambda_hat (one high-precision exponential per row), omega_hat ----------------
  double lw[4];
  float omh[4];
  bool big = false;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    lam[a] = isinf(st.mu[a]) ? 0.0f : (float)exp((double)__fsub_rn(st.mu[a], muh[a]));
    lw[a] = __dmul_rn((double)lam[a], (double)st.om[a]);
    double R = (own8 ? rs8[a] : 0.0) + rs16[a];
    R += shfl_xor_d(R, 1);
    R += shfl_xor_d(R, 2);
    big |= !(R < 4096.0);
    omh[a] = (float)__dadd_rn(lw[a], R);
  }

  // ---- stage 2: block-LAMP problem, eq. (8) ---------------------------------------------
  const uint32_t freem = actmask & ~Theta;
  uint32_t Rset = 0;
  if (!force8 && !force16 && freem) {
    double xi[4] = {0.0, 0.0, 0.0, 0.0};
    if (own8) {
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const double oh = (double)omh[a];
#pragma unroll
        for (int b = 0; b < 16; ++b) {
          // invisible pairs hold e = 0 and add exactly +0
          const double e = (double)acc[a][b];
          xi[a] = __dadd_rn(xi[a], __dmul_rn(__dsub_rn(oh, e), e));
        }
      }
    }
    uint32_t feas = 0xffffu;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      double x[4];
#pragma unroll
      for (int th = 0; th < 4; ++th) x[th] = shfl_d(xi[a], (lane & ~3) | th);
      const double oh = (double)omh[a];
      const double rhs = __dmul_rn(__dmul_rn((double)P.tau, oh), oh);
#pragma unroll
      for (uint32_t r = 0; r < 16; ++r) {
        const uint32_t keep = freem & ~r;
        double kept = 0.0;
#pragma unroll
        for (int th = 0; th < 4; ++th)
          if ((keep >> th) & 1u) kept = __dadd_rn(kept, x[th]);
        if (!(kept <= rhs)) feas &= ~(1u << r);
      }
    }
    feas = __reduce_and_sync(kFull, feas);
    // smallest recompute set, then smallest bitmask, among subsets of the free sub-blocks
    int best = 5;
#pragma unroll
    for (uint32_t r = 0; r < 16; ++r) {
      const int sz = __popc(r);
      if ((r & ~freem) == 0 && ((feas >> r) & 1u) && sz < best) { best = sz; Rset = r; }
    }
  }

  // ---- stage-2 recomputation with the maxima unchanged ---------------------------------
  for (int th = 0; th < 4; ++th) {
    if (!((Rset >> th) & 1u)) continue;
    float y[4][4];
    dot16<D>(kf, qrow, P.qs[2], th, th_own, scale_d, y);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        es_lane[(16 * th + b) * kBQ + a] = y[a][b];
        if (vis<FULL>(g, 16 * th + 4 * th_own + b, 4 * qa + a)) wc.sat16 += fabsf(y[a][b]) == 448.0f;
      }
    exp_block(th);
  }

  // ---- state update ----------------------------------------------------------------------
  const bool keep8 = own8 && !((Rset >> th_own) & 1u);
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    double R = (keep8 ? rs8[a] : 0.0) + rs16[a];
    R += shfl_xor_d(R, 1);
    R += shfl_xor_d(R, 2);
    big |= !(R < 4096.0);
    st.mu[a] = muh[a];
    st.om[a] = (float)__dadd_rn(lw[a], R);
  }
  // the 8-bit exponentials that stay (and zeros of inactive sub-blocks) join the tile
  if (keep8 || !own_act) {
    float* dst = es + (16 * th_own) * kBQ + 4 * qa;
#pragma unroll
    for (int b = 0; b < 16; ++b)
      *reinterpret_cast<float4*>(dst + b * kBQ) = make_float4(acc[0][b], acc[1][b], acc[2][b], acc[3][b]);
  }

  if (__any_sync(kFull, big)) wc.bigrow++;
  wc.active += nact;
  wc.s1 += __popc(Theta);
  wc.s2 += __popc(Rset);
  wc.hist[__popc(Theta | Rset)]++;
  return Theta | (Rset << 4);
}

}  // namespace lamp
