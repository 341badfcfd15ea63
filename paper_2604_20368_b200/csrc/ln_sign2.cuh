// Fused sign pass of the kernel gradient (App. A): both gradients of one kernel block in one sweep.
//
// For a block A_ij = k(x_i, y_j) with upstream g_ij = dA_ij * A_ij / lambda,
//     rows[i][c]        = - sum_j              g_ij sign(x_ic - y_jc)          (gradient w.r.t. the tokens x)
//     part[chunk][j][c] = + sum_{i in chunk}   g_ij sign(x_ic - y_jc)          (gradient w.r.t. the landmarks y)
// with sign(0) = 0.  Both sums share the difference t = x - y and the step h = half_step(t); per
// (pair, dim) the FMA pipe sees one packed subtract, one saturating multiply-add and two packed
// multiply-adds (4 lane-operations; two separate passes cost 6).
//
// grid (chunks, D/64, heads); block (16, TG), TG even, <= 16.  Thread (tc, tt) owns 8 tokens
// (tt*8 .. tt*8+7 of the current token tile) and 4 dims (tc*4 .. tc*4+3 of the CTA's 64-dim slab).
// Row sums stay in registers over all landmarks.  Column sums are partial over a thread's 8 tokens:
// per landmark every thread leaves 4 values in shared memory, and after each round of 4 landmarks
// the CTA adds the TG partials of each (landmark, dim), in a fixed order, into an accumulator in
// shared memory that lives as long as the CTA's token chunk.  The landmark and g tiles of the next
// round are fetched into registers while the current round is computed (two buffers, one barrier
// per round).  sum_j g_ij and sum_i g_ij, which the step formulation needs, come from the threads
// that load the g tile.
#pragma once
#include "ln_common.cuh"

namespace ln {

constexpr int S2_RL = 4;       // landmarks per round
constexpr int S2_DS = 64;      // dims per CTA

struct Sign2Smem {             // offsets in floats into the dynamic shared memory
  int cacc, colsum, cp, ls, gs2, rowsum, cw, total;
};
__host__ __device__ inline Sign2Smem sign2_smem(int m, int TG) {
  const int mr = (m + S2_RL - 1) / S2_RL * S2_RL;
  Sign2Smem s; int o = 0;
  s.cacc = o;   o += mr * S2_DS;
  s.cp = o;     o += 2 * S2_RL * 16 * S2_DS;     // 16 group slots whatever TG is: the sum over groups is unrolled
  s.gs2 = o;    o += 2 * S2_RL * 8 * TG * 2;
  s.ls = o;     o += 2 * S2_RL * S2_DS;
  s.colsum = o; o += mr;
  s.rowsum = o; o += 2 * 8 * TG;
  s.cw = o;     o += 2 * 4 * S2_RL;
  s.total = o;
  return s;
}

template <typename TT, typename TO>
__global__ void __launch_bounds__(256, 2) k_sign2(const TT* __restrict__ tok, const float* __restrict__ Lm,
                                                  const float* __restrict__ G, int ldg, TO* __restrict__ rows,
                                                  float* __restrict__ part, int n, int m, int D, int rpc) {
  extern __shared__ __align__(16) float s2_smem[];
  const int TG = blockDim.y, tc = threadIdx.x, tt = threadIdx.y;
  const int tid = tt * 16 + tc, nthr = 16 * TG, TT8 = 8 * TG, warp = tid >> 5, lane = tid & 31;
  const int chunk = blockIdx.x, slab = blockIdx.y, bh = blockIdx.z, nchunks = gridDim.x;
  const Sign2Smem so = sign2_smem(m, TG);
  float* Cacc = s2_smem + so.cacc;
  float* Cp = s2_smem + so.cp;                                      // [2][RL][16][64]; slots >= TG stay zero
  f32x2* Gs2 = reinterpret_cast<f32x2*>(s2_smem + so.gs2);          // [2][RL][8 TG] pairs (g, g)
  float* Ls = s2_smem + so.ls;                                      // [2][RL][64], negated
  float* colsum = s2_smem + so.colsum;
  float* rowsum = s2_smem + so.rowsum;                              // [2][8 TG]
  float* cw = s2_smem + so.cw;                                      // [2][4 warps][RL]
  tok += (long long)bh * n * D + slab * S2_DS;
  Lm += (long long)bh * m * D + slab * S2_DS;
  G += (long long)bh * n * ldg;
  rows += (long long)bh * n * D + slab * S2_DS;
  const int ibeg = chunk * rpc, iend = min(n, ibeg + rpc);
  const int nrounds = (m + S2_RL - 1) / S2_RL, mr = nrounds * S2_RL;
  const int ntiles = (iend - ibeg + TT8 - 1) / TT8, total = ntiles * nrounds;
  const bool gvec = (ldg & 3) == 0;
  const int lwarps = (TT8 + 31) >> 5;           // warps that hold loader threads of the g tile

  for (int e = tid; e < mr * S2_DS; e += nthr) Cacc[e] = 0.f;
  for (int e = tid; e < 2 * S2_RL * 16 * S2_DS; e += nthr) Cp[e] = 0.f;
  for (int e = tid; e < mr; e += nthr) colsum[e] = 0.f;

  float rs = 0.f;                               // loader: sum_j g_ij of this thread's token over the rounds of a tile
  // global -> registers: g of (token tid of the tile, 4 landmarks of the round), one 4-dim piece of the landmark tile
  auto fetch = [&](int tile, int r, float4& gq, float4& lq) {
    const int l0 = r * S2_RL;
    gq = make_float4(0.f, 0.f, 0.f, 0.f); lq = gq;
    const int i = ibeg + tile * TT8 + tid;
    if (tid < TT8 && i < iend) {
      const float* gp = G + (long long)i * ldg + l0;
      if (gvec) gq = *reinterpret_cast<const float4*>(gp);
      else { gq.x = gp[0]; if (l0 + 1 < m) gq.y = gp[1]; if (l0 + 2 < m) gq.z = gp[2]; if (l0 + 3 < m) gq.w = gp[3]; }
      if (l0 + 1 >= m) gq.y = 0.f;
      if (l0 + 2 >= m) gq.z = 0.f;
      if (l0 + 3 >= m) gq.w = 0.f;
    }
    if (tid < S2_RL * 16) {
      const int l = l0 + (tid >> 4);
      if (l < m) lq = *reinterpret_cast<const float4*>(Lm + (long long)l * D + (tid & 15) * 4);
    }
  };
  // registers -> shared memory of buffer it & 1, plus the row / column sums of g
  auto stash = [&](int buf, int tile, int r, const float4& gq, const float4& lq) {
    if (tid < TT8) {
      f32x2* g2 = Gs2 + (size_t)buf * S2_RL * TT8 + tid;
      g2[0] = pack2(gq.x, gq.x); g2[TT8] = pack2(gq.y, gq.y); g2[2 * TT8] = pack2(gq.z, gq.z); g2[3 * TT8] = pack2(gq.w, gq.w);
      if (r == 0) rs = 0.f;
      rs += (gq.x + gq.y) + (gq.z + gq.w);
      if (r == nrounds - 1) rowsum[(tile & 1) * TT8 + tid] = rs;
    }
    if (tid < S2_RL * 16)
      *reinterpret_cast<float4*>(Ls + buf * S2_RL * S2_DS + (tid >> 4) * S2_DS + (tid & 15) * 4) = make_float4(-lq.x, -lq.y, -lq.z, -lq.w);
    if (warp < lwarps) {                        // column sums of the g tile over this warp's 32 tokens
      float c0 = gq.x, c1 = gq.y, c2 = gq.z, c3 = gq.w;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        c0 += __shfl_xor_sync(0xffffffffu, c0, o); c1 += __shfl_xor_sync(0xffffffffu, c1, o);
        c2 += __shfl_xor_sync(0xffffffffu, c2, o); c3 += __shfl_xor_sync(0xffffffffu, c3, o);
      }
      if (lane == 0) *reinterpret_cast<float4*>(cw + (buf * 4 + warp) * S2_RL) = make_float4(c0, c1, c2, c3);
    }
  };
  // the column sums of round `it` (left in cw by stash) join the running sums
  auto fold_colsum = [&](int buf, int r) {
    if (tid < S2_RL) {
      float s = 0.f;
      for (int w = 0; w < lwarps; ++w) s += cw[(buf * 4 + w) * S2_RL + tid];
      colsum[r * S2_RL + tid] += s;
    }
  };

  {
    float4 gq, lq;
    if (total > 0) { fetch(0, 0, gq, lq); stash(0, 0, 0, gq, lq); }
  }
  __syncthreads();
  if (total > 0) fold_colsum(0, 0);

  f32x2 qp[8][2], accR[8][2];
  int tile = 0, r = 0;
  for (int it = 0; it < total; ++it) {
    const int buf = it & 1;
    int tile_n = tile, r_n = r + 1;               // the round after this one
    if (r_n == nrounds) { r_n = 0; ++tile_n; }
    float4 gq, lq;
    const bool more = it + 1 < total;
    if (more) fetch(tile_n, r_n, gq, lq);
    if (r == 0) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = ibeg + tile * TT8 + tt * 8 + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < iend) v = ld4(tok + (long long)i * D + tc * 4);
        qp[k][0] = pack2(v.x, v.y); qp[k][1] = pack2(v.z, v.w);
        accR[k][0] = 0ull; accR[k][1] = 0ull;
      }
    }
    const f32x2* g2 = Gs2 + (size_t)buf * S2_RL * TT8 + tt * 8;
    const float* ls = Ls + buf * S2_RL * S2_DS + tc * 4;
    float* cp = Cp + ((size_t)(buf * S2_RL) * 16 + tt) * S2_DS + tc * 4;
#pragma unroll
    for (int jj = 0; jj < S2_RL; ++jj) {
      const ulonglong2 nl = *reinterpret_cast<const ulonglong2*>(ls + jj * S2_DS);
      f32x2 gg[8];
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(g2 + jj * TT8 + 2 * k2);
        gg[2 * k2] = t.x; gg[2 * k2 + 1] = t.y;
      }
      f32x2 c0a = 0ull, c1a = 0ull, c0b = 0ull, c1b = 0ull;     // two chains per dim pair
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const f32x2 t0 = add2(qp[k][0], nl.x), t1 = add2(qp[k][1], nl.y);
        const f32x2 h0 = pack2(half_step(lo32(t0)), half_step(hi32(t0)));
        const f32x2 h1 = pack2(half_step(lo32(t1)), half_step(hi32(t1)));
        accR[k][0] = fma2(gg[k], h0, accR[k][0]);
        accR[k][1] = fma2(gg[k], h1, accR[k][1]);
        if (k & 1) { c0b = fma2(gg[k], h0, c0b); c1b = fma2(gg[k], h1, c1b); }
        else       { c0a = fma2(gg[k], h0, c0a); c1a = fma2(gg[k], h1, c1a); }
      }
      ulonglong2 cs; cs.x = add2(c0a, c0b); cs.y = add2(c1a, c1b);
      *reinterpret_cast<ulonglong2*>(cp + jj * 16 * S2_DS) = cs;
    }
    if (r == nrounds - 1) {                     // all landmarks seen: rows of this token tile
      const float* rsum = rowsum + (tile & 1) * TT8 + tt * 8;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int i = ibeg + tile * TT8 + tt * 8 + k;
        if (i < iend) {
          const float gs = rsum[k];
          st4(rows + (long long)i * D + tc * 4, make_float4(gs - 2.f * lo32(accR[k][0]), gs - 2.f * hi32(accR[k][0]),
                                                            gs - 2.f * lo32(accR[k][1]), gs - 2.f * hi32(accR[k][1])));
        }
      }
    }
    if (more) stash(buf ^ 1, tile_n, r_n, gq, lq);
    __syncthreads();
    // column partials of this round -> accumulator (fixed order over the token groups)
    for (int o = tid; o < S2_RL * S2_DS; o += nthr) {
      const float* src = Cp + (buf * S2_RL + (o >> 6)) * 16 * S2_DS + (o & 63);
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
      for (int g = 0; g < 16; g += 4) {
        s0 += src[g * S2_DS]; s1 += src[(g + 1) * S2_DS]; s2 += src[(g + 2) * S2_DS]; s3 += src[(g + 3) * S2_DS];
      }
      Cacc[(r * S2_RL + (o >> 6)) * S2_DS + (o & 63)] += (s0 + s1) + (s2 + s3);
    }
    if (more) fold_colsum(buf ^ 1, r_n);
    tile = tile_n; r = r_n;
  }
  __syncthreads();
  float* outp = part + ((long long)bh * nchunks + chunk) * m * D + slab * S2_DS;
  for (int e = tid; e < m * S2_DS; e += nthr) {
    const int l = e >> 6, c = e & 63;
    outp[(long long)l * D + c] = 2.f * Cacc[e] - colsum[l];
  }
}

}  // namespace ln
