// Fused sign pass of the kernel gradient (App. A): both gradients of one kernel block in one sweep.
//
// For a block A_ij = k(x_i, y_j) with upstream g_ij = dA_ij * A_ij / lambda,
//     rows[i][c]        = - sum_j              g_ij sign(x_ic - y_jc)          (gradient w.r.t. the tokens x)
//     part[chunk][j][c] = + sum_{i in chunk}   g_ij sign(x_ic - y_jc)          (gradient w.r.t. the landmarks y)
// with sign(0) = 0.  Both sums share the step h = (sign(x - y) + 1) / 2; per (pair, dim) the FMA pipe sees
// one saturating multiply-add and two packed multiply-adds (3 lane-operations), plus one packed
// subtract where the tokens are fp32 (two separate passes cost 6).
//
// bf16 tokens: the subtraction is folded into the saturating multiply-add.  For a landmark value y with
// exponent e (y = +-1.f * 2^e) take s = 2^(22 - e) and b = -y s + 1/2: |y| s lies in [2^22, 2^23), where
// the spacing of fp32 is 1/2, so b is exact, and  h = sat(fma(x, s, b)) = sat(round((x - y) s + 1/2)).
// A bf16 x that differs from y differs by at least one unit in the last place of y (x - y is a multiple
// of the smaller of the two spacings, and bf16's is the larger unless x is 2^16 times smaller than y),
// so (x - y) s is 0 or at least 1/2 in magnitude: h is exactly 0, 1/2 or 1.  y = 0 (and |y| < 2^-104)
// take s = 2^126.  The pairs (s, b) are formed once per landmark tile by the threads that load it.
//
// grid (chunks, D/64, heads); block (16, TG), TG even, 8 <= TG <= 16.  Thread (tc, tt) owns 8 tokens
// (tt*8 .. tt*8+7 of the current token tile) and 4 dims (4 tc .. 4 tc + 3 of the CTA's 64-dim slab).
// Row sums stay in registers over all landmarks.  Column sums are partial over a thread's 8 tokens:
// per landmark every thread leaves 4 values in shared memory, and after each round of 8 landmarks
// the CTA adds the TG partials of each (landmark, dim), in a fixed order, into the running sums,
// which live in the output array itself (global memory; each element belongs to one thread, which
// reads it at the start of a round and writes it at the end).  The landmark and g tiles of the next
// round are fetched into registers while the current round is computed (two buffers, one barrier
// per round).  sum_j g_ij comes from the threads that load the g tile, sum_i g_ij from the g tile in
// shared memory.  All shared-memory strides are compile-time constants.
#pragma once
#include "ln_common.cuh"

namespace ln {

constexpr int S2_RL = 8;        // landmarks per round
constexpr int S2_DS = 64;       // dims per CTA
constexpr int S2_TGMAX = 16;    // token groups per CTA
constexpr int S2_TOK = 8 * S2_TGMAX;
// shared memory, in floats
constexpr int S2_CP = 0;                                           // [2][RL][TGMAX][64] column partials
constexpr int S2_GS = S2_CP + 2 * S2_RL * S2_TGMAX * S2_DS;        // [2][RL][TOK] pairs (g, g)
constexpr int S2_LS = S2_GS + 2 * S2_RL * S2_TOK * 2;              // [2][RL][2][64]: negated landmark values, or scales s and offsets b
constexpr int S2_LROW = 2 * S2_DS;
constexpr int S2_RS = S2_LS + 2 * S2_RL * S2_LROW;                 // [2][TOK] row sums of g
constexpr int S2_CS = S2_RS + 2 * S2_TOK;                          // [mr] column sums of g over the chunk
__host__ __device__ inline size_t sign2_smem_bytes(int m) { return sizeof(float) * (size_t)(S2_CS + (m + S2_RL - 1) / S2_RL * S2_RL); }

// NR = float2 column outputs per thread and round: 1 with 256 threads, 2 with 128 .. 254.
template <typename TT, typename TO, int NR>
__global__ void __launch_bounds__(256, 2) k_sign2(const TT* __restrict__ tok, const float* __restrict__ Lm,
                                                  const float* __restrict__ G, int ldg, TO* __restrict__ rows,
                                                  float* __restrict__ part, int n, int m, int D, int rpc) {
  extern __shared__ __align__(16) float s2_smem[];
  const int TG = blockDim.y, tc = threadIdx.x, tt = threadIdx.y;
  const int tid = tt * 16 + tc, nthr = 16 * TG, TT8 = 8 * TG, warp = tid >> 5, lane = tid & 31, nwarps = nthr >> 5;
  const int chunk = blockIdx.x, slab = blockIdx.y, bh = blockIdx.z, nchunks = gridDim.x;
  float* const Cp = s2_smem + S2_CP;
  f32x2* const Gs = reinterpret_cast<f32x2*>(s2_smem + S2_GS);
  float* const Ls = s2_smem + S2_LS;
  float* const rowsum = s2_smem + S2_RS;
  float* const colsum = s2_smem + S2_CS;
  tok += (long long)bh * n * D + slab * S2_DS + 4 * tc;
  rows += (long long)bh * n * D + slab * S2_DS + 4 * tc;
  float* const outp = part + ((long long)bh * nchunks + chunk) * m * D + slab * S2_DS;
  const int ibeg = chunk * rpc, iend = min(n, ibeg + rpc);
  const int nrounds = (m + S2_RL - 1) / S2_RL, mr = nrounds * S2_RL;
  const int ntiles = (iend - ibeg + TT8 - 1) / TT8, total = ntiles * nrounds;
  const bool gvec = (ldg & 3) == 0;

  // group slots >= TG of the column partials are never written: they are zeroed once, the sum over slots is unrolled
  for (int e = tid; e < 2 * S2_RL * (S2_TGMAX - TG) * S2_DS; e += nthr) {
    const int row = e / ((S2_TGMAX - TG) * S2_DS), rest = e % ((S2_TGMAX - TG) * S2_DS);
    Cp[row * (S2_TGMAX * S2_DS) + TG * S2_DS + rest] = 0.f;
  }
  for (int e = tid; e < mr; e += nthr) colsum[e] = 0.f;
  if (total == 0) {
    for (int e = tid; e < m * S2_DS; e += nthr) outp[(long long)(e >> 6) * D + (e & 63)] = 0.f;
    return;
  }
  // loader roles.  g tile: thread tid fetches g of (token tid / 2 of the tile, landmarks 4 (tid & 1) .. + 3 of the
  // round): 16 TG = nthr pieces.  Landmark tile: the last 128 threads fetch one 4-dim piece each.
  const int ltok = tid >> 1, lhalf = tid & 1;
  const int lpiece = tid - (nthr - 128);
  const float* gsrc = G + ((long long)bh * n + ibeg + ltok) * ldg + 4 * lhalf;        // this thread's g row, round 0
  const float* lsrc = Lm + (long long)bh * m * D + slab * S2_DS + (lpiece >> 4) * D + (lpiece & 15) * 4;
  const int gdst = lhalf * 4 * S2_TOK + ltok;                      // f32x2 index inside one buffer of Gs
  const int ldst = (lpiece >> 4) * S2_LROW + (lpiece & 15) * 4;    // float index inside one buffer of Ls
  constexpr bool FOLD = sizeof(TT) == 2;                           // bf16 tokens: subtraction folded into the step
  float rs = 0.f;                                                  // sum over the rounds of a tile of this thread's g values

  // fetch of the round the pointers stand at; tok_ok: this thread's token of that tile is inside the chunk
  const float* gp = gsrc;
  const float* lp = lsrc;
  auto fetch = [&](int tile, int r, float4& gq, float4& lq) {
    gq = make_float4(0.f, 0.f, 0.f, 0.f); lq = gq;
    const int lg = r * S2_RL + 4 * lhalf;
    if (ibeg + tile * TT8 + ltok < iend && lg < m) {
      if (gvec) gq = *reinterpret_cast<const float4*>(gp);
      else { gq.x = gp[0]; if (lg + 1 < m) gq.y = gp[1]; if (lg + 2 < m) gq.z = gp[2]; if (lg + 3 < m) gq.w = gp[3]; }
      if (lg + 1 >= m) gq.y = 0.f;
      if (lg + 2 >= m) gq.z = 0.f;
      if (lg + 3 >= m) gq.w = 0.f;
    }
    if (lpiece >= 0 && r * S2_RL + (lpiece >> 4) < m) lq = *reinterpret_cast<const float4*>(lp);
  };
  const long long g_tile_step = (long long)TT8 * ldg - (long long)(nrounds - 1) * S2_RL;   // last round of a tile -> round 0 of the next
  const long long l_wrap = (long long)(nrounds - 1) * S2_RL * D;
  auto stash = [&](int buf, int tile, int r, const float4& gq, const float4& lq) {
    f32x2* g2 = Gs + buf * (S2_RL * S2_TOK) + gdst;
    g2[0] = pack2(gq.x, gq.x); g2[S2_TOK] = pack2(gq.y, gq.y); g2[2 * S2_TOK] = pack2(gq.z, gq.z); g2[3 * S2_TOK] = pack2(gq.w, gq.w);
    if (lpiece >= 0) {
      float* ld = Ls + buf * (S2_RL * S2_LROW) + ldst;
      if constexpr (FOLD) {
        float4 sc, of;
        fold_pair(lq.x, sc.x, of.x); fold_pair(lq.y, sc.y, of.y); fold_pair(lq.z, sc.z, of.z); fold_pair(lq.w, sc.w, of.w);
        *reinterpret_cast<float4*>(ld) = sc;
        *reinterpret_cast<float4*>(ld + S2_DS) = of;
      } else {
        *reinterpret_cast<float4*>(ld) = make_float4(-lq.x, -lq.y, -lq.z, -lq.w);
      }
    }
    if (r == 0) rs = 0.f;
    rs += (gq.x + gq.y) + (gq.z + gq.w);
    if (r == nrounds - 1) {
      const float both = rs + __shfl_xor_sync(0xffffffffu, rs, 1);
      if (lhalf == 0) rowsum[(tile & 1) * S2_TOK + ltok] = both;
    }
  };
  // column sums of the g tile in buffer `buf` (round r) join the running sums: warp w takes landmarks w, w + nwarps, ...
  auto fold_colsum = [&](int buf, int r) {
    for (int jj = warp; jj < S2_RL; jj += nwarps) {
      const f32x2* g2 = Gs + buf * (S2_RL * S2_TOK) + jj * S2_TOK;
      float s = 0.f;
#pragma unroll
      for (int q = 0; q < S2_TOK / 32; ++q) { const int t = lane + 32 * q; if (t < TT8) s += lo32(g2[t]); }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) colsum[r * S2_RL + jj] += s;
    }
  };

  {
    float4 gq, lq;
    fetch(0, 0, gq, lq); stash(0, 0, 0, gq, lq);
  }
  __syncthreads();

  // column outputs of a round: 8 landmarks x 64 dims = 256 float2; thread o takes landmark o / 32, dims 2 (o % 32)
  int cjj[NR], coff[NR], csrc[NR];
#pragma unroll
  for (int u = 0; u < NR; ++u) {
    const int o = tid + u * nthr;
    cjj[u] = (o < S2_RL * 32) ? (o >> 5) : (1 << 20);          // out of range -> never below the landmarks left
    coff[u] = (o >> 5) * D + 2 * (o & 31);
    csrc[u] = (o >> 5) * (S2_TGMAX * S2_DS) + 2 * (o & 31);
  }
  // The column partials of a round are added up while the NEXT round computes (their loads and adds are spread
  // over its instruction stream), so that no phase of a round leaves the FMA pipe without work.
  int red_buf = 0, red_mleft = 0, red_r = 0;    // the round whose partials are pending (red_mleft = 0: none)
  bool red_last = false, red_first = true;
  float* red_out = outp;
  float* outr = outp;                           // outputs of the current round: outp + r * RL * D
  f32x2 qp[8][2], accR[8][2];
  int tile = 0, r = 0;
  for (int it = 0; it < total; ++it) {
    const int buf = it & 1;
    int tile_n = tile, r_n = r + 1;             // the round after this one
    if (r_n == nrounds) { r_n = 0; ++tile_n; gp += g_tile_step; lp -= l_wrap; }
    else { gp += S2_RL; lp += S2_RL * D; }
    float4 gq, lq;
    const bool more = it + 1 < total;
    if (more) fetch(tile_n, r_n, gq, lq);
    float2 pend[NR], pend2[NR];                 // pending round: running sums of earlier tiles, then + partials
#pragma unroll
    for (int u = 0; u < NR; ++u) {
      pend[u] = (!red_first && cjj[u] < red_mleft) ? *reinterpret_cast<const float2*>(red_out + coff[u]) : make_float2(0.f, 0.f);
      pend2[u] = make_float2(0.f, 0.f);
    }
    if (r == 0) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = ibeg + tile * TT8 + tt * 8 + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < iend) v = ld4(tok + (long long)i * D);
        qp[k][0] = pack2(v.x, v.y); qp[k][1] = pack2(v.z, v.w);
        accR[k][0] = 0ull; accR[k][1] = 0ull;
      }
    }
    const f32x2* g2 = Gs + buf * (S2_RL * S2_TOK) + tt * 8;
    const float* ls = Ls + buf * (S2_RL * S2_LROW) + tc * 4;
    float* cp = Cp + buf * (S2_RL * S2_TGMAX * S2_DS) + tt * S2_DS + tc * 4;
    const float* rsrc = Cp + red_buf * (S2_RL * S2_TGMAX * S2_DS);
#pragma unroll
    for (int jj = 0; jj < S2_RL; ++jj) {
      if ((jj & 1) == 0) {                      // a quarter of the pending round's partial sums
#pragma unroll
        for (int u = 0; u < NR; ++u)
          if (cjj[u] < red_mleft) {
            const float* src = rsrc + csrc[u] + (jj * 2) * S2_DS;
            const float2 a0 = *reinterpret_cast<const float2*>(src), a1 = *reinterpret_cast<const float2*>(src + S2_DS);
            const float2 a2 = *reinterpret_cast<const float2*>(src + 2 * S2_DS), a3 = *reinterpret_cast<const float2*>(src + 3 * S2_DS);
            pend[u].x += a0.x; pend[u].y += a0.y; pend2[u].x += a1.x; pend2[u].y += a1.y;
            pend[u].x += a2.x; pend[u].y += a2.y; pend2[u].x += a3.x; pend2[u].y += a3.y;
          }
      }
      if (jj == 1) fold_colsum(buf, r);         // column sums of this round's g tile
      const ulonglong2 nl = *reinterpret_cast<const ulonglong2*>(ls + jj * S2_LROW);
      float4 ob = make_float4(0.f, 0.f, 0.f, 0.f);
      if constexpr (FOLD) ob = *reinterpret_cast<const float4*>(ls + jj * S2_LROW + S2_DS);
      f32x2 gg[8];
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(g2 + jj * S2_TOK + 2 * k2);
        gg[2 * k2] = t.x; gg[2 * k2 + 1] = t.y;
      }
      f32x2 c0 = 0ull, c1 = 0ull;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        f32x2 h0, h1;
        if constexpr (FOLD) {
          h0 = pack2(sat_fma(lo32(qp[k][0]), lo32(nl.x), ob.x), sat_fma(hi32(qp[k][0]), hi32(nl.x), ob.y));
          h1 = pack2(sat_fma(lo32(qp[k][1]), lo32(nl.y), ob.z), sat_fma(hi32(qp[k][1]), hi32(nl.y), ob.w));
        } else {
          const f32x2 t0 = add2(qp[k][0], nl.x), t1 = add2(qp[k][1], nl.y);
          h0 = pack2(half_step(lo32(t0)), half_step(hi32(t0)));
          h1 = pack2(half_step(lo32(t1)), half_step(hi32(t1)));
        }
        accR[k][0] = fma2(gg[k], h0, accR[k][0]);
        accR[k][1] = fma2(gg[k], h1, accR[k][1]);
        c0 = fma2(gg[k], h0, c0);
        c1 = fma2(gg[k], h1, c1);
      }
      ulonglong2 cs; cs.x = c0; cs.y = c1;
      *reinterpret_cast<ulonglong2*>(cp + jj * (S2_TGMAX * S2_DS)) = cs;
    }
#pragma unroll
    for (int u = 0; u < NR; ++u)
      if (cjj[u] < red_mleft) {
        float2 v = make_float2(pend[u].x + pend2[u].x, pend[u].y + pend2[u].y);
        if (red_last) { const float cs = colsum[red_r * S2_RL + cjj[u]]; v.x = 2.f * v.x - cs; v.y = 2.f * v.y - cs; }
        *reinterpret_cast<float2*>(red_out + coff[u]) = v;
      }
    if (r == nrounds - 1) {                     // all landmarks seen: rows of this token tile
      const float* rsum = rowsum + (tile & 1) * S2_TOK + tt * 8;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = ibeg + tile * TT8 + tt * 8 + k;
        if (i < iend) {
          const float gs = rsum[k];
          st4(rows + (long long)i * D, make_float4(gs - 2.f * lo32(accR[k][0]), gs - 2.f * hi32(accR[k][0]),
                                                   gs - 2.f * lo32(accR[k][1]), gs - 2.f * hi32(accR[k][1])));
        }
      }
    }
    if (more) stash(buf ^ 1, tile_n, r_n, gq, lq);
    __syncthreads();
    red_buf = buf; red_mleft = m - r * S2_RL; red_r = r; red_last = tile == ntiles - 1; red_first = tile == 0; red_out = outr;
    if (r_n == 0) outr = outp; else outr += S2_RL * D;
    tile = tile_n; r = r_n;
  }
  // the last round's partials
#pragma unroll
  for (int u = 0; u < NR; ++u)
    if (cjj[u] < red_mleft) {
      const float* src = Cp + red_buf * (S2_RL * S2_TGMAX * S2_DS) + csrc[u];
      float2 s0 = red_first ? make_float2(0.f, 0.f) : *reinterpret_cast<const float2*>(red_out + coff[u]), s1 = make_float2(0.f, 0.f);
#pragma unroll
      for (int g = 0; g < S2_TGMAX; g += 2) {
        const float2 a = *reinterpret_cast<const float2*>(src + g * S2_DS), b2 = *reinterpret_cast<const float2*>(src + (g + 1) * S2_DS);
        s0.x += a.x; s0.y += a.y; s1.x += b2.x; s1.y += b2.y;
      }
      const float cs = colsum[red_r * S2_RL + cjj[u]];
      *reinterpret_cast<float2*>(red_out + coff[u]) = make_float2(2.f * (s0.x + s1.x) - cs, 2.f * (s0.y + s1.y) - cs);
    }
}

}  // namespace ln
