// FP32 CUDA-core kernels of the Laplacian-Nystrom path.  Every kernel works on one
// (batch*head) slice per blockIdx.z / blockIdx.y and a tile of tokens or landmarks per
// blockIdx.x.  All intermediates are fp32; only the [.,.,.,d] user tensors have a storage type.
#pragma once
#include "ln_common.cuh"
#include "ln_mma.cuh"
#include "ln_ns_umma.cuh"
#include "ln_ns_umma256.cuh"
#include "ln_gemm_umma.cuh"

namespace ln {

// =====================================================================================
// Laplacian kernel block (Sec. 1, Eq. 8):  E[i][j] = exp(-sum_c |a_ic - b_jc| / lambda)
//
// Block = (LG, TG) threads: thread (tj, ti) owns the 8 x 4 pairs of tokens ti + TG*k (k < 8) and
// landmarks tj + LG*q (q < 4) of a (8 TG) x (4 LG) tile, so the tile follows the problem size
// (n = 197, m = 49 run as one 200 x 52 tile per head instead of two 128 x 64 tiles).  Operands
// are staged in shared memory token-major as fp32 in chunks of 32 dims straight from coalesced
// 16-byte global loads (no transpose); a thread reads four dims of a row with one 128-bit load.
// Per (pair, dim) the work is two FP32 instructions: subtract, add |.|.
// Up to three problems that share the landmark operand (C = k(Q,L), R^T = k(K,L), W = k(L,L)) go
// in one launch (blockIdx.z).
// =====================================================================================
constexpr int L1_DC = 32;            // dims per staged chunk
constexpr int L1_PITCH = L1_DC + 4;  // floats per staged row

struct L1Prob {
  const void* A; float* E; float* rowsum;
  long long sA, sE;      // per-batch strides of A (elements) and E
  int na, lde, a_f32;
  float rs_scale;
  double* stat;          // NULL, or column statistics of E per token tile: [batch][tiles][nb][2] = (sum_i E_ij, sum_i E_ij^2)
};
struct L1Args {
  L1Prob p[3];
  const void* Bm; long long sB;
  int nb, d, b_f32;
  float nscale;          // -log2(e) / lambda
  int jsplits = 1;       // > 1 (one problem, no row sums or statistics): blockIdx.z splits the landmark range instead of naming a problem
};

// 8 consecutive elements of a row -> fp32 (zero outside [0, d)); vec: the row start is 16-byte aligned
__device__ __forceinline__ void l1_fetch8(const void* base, bool f32, long long row_off, int c, int d, bool vec, float (&v)[8]) {
  if (f32) {
    const float* p = reinterpret_cast<const float*>(base) + row_off + c;
    if (vec && c + 8 <= d) {
      const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = (c + q < d) ? p[q] : 0.f;
    }
  } else {
    const bf16* p = reinterpret_cast<const bf16*>(base) + row_off + c;
    if (vec && c + 8 <= d) {
      const uint4 r = *reinterpret_cast<const uint4*>(p);
      const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) { v[2 * q] = __uint_as_float(w[q] << 16); v[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u); }
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = (c + q < d) ? __bfloat162float(p[q]) : 0.f;
    }
  }
}

// QN = landmarks per thread: 4 (128 registers, two CTAs per SM) for large problems; 2 (three CTAs per
// SM) where a CTA lives too briefly for two of them to hide each other's loads and epilogues.
template <int QN>
__global__ void __launch_bounds__(256, QN == 4 ? 2 : 3) k_l1(const L1Args args) {
  extern __shared__ __align__(16) float l1_smem[];
  const L1Prob pr = args.p[args.jsplits > 1 ? 0 : blockIdx.z];
  const int LG = blockDim.x, TG = blockDim.y, tj = threadIdx.x, ti = threadIdx.y;
  const int tid = ti * LG + tj, nthr = LG * TG;
  const int TA = 8 * TG, TB = QN * LG;
  const int i0 = blockIdx.x * TA, b = blockIdx.y;
  if (i0 >= pr.na) return;
  float* As = l1_smem;                    // [TA][L1_PITCH]
  float* Bs = l1_smem + TA * L1_PITCH;    // [TB][L1_PITCH]
  float* Rs = Bs + TB * L1_PITCH;         // [TA][LG] row-sum partials
  const int na = pr.na, nb = args.nb, d = args.d, lde = pr.lde;
  const bool vec = (d % 8) == 0;
  float* E = pr.E + (long long)b * pr.sE;
  float rs[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) rs[k] = 0.f;

  // landmark tiles of this CTA: all of them, or its share of a split range (whole tiles)
  const int jper = args.jsplits > 1 ? ((nb + args.jsplits - 1) / args.jsplits + TB - 1) / TB * TB : nb;
  const int jbeg = args.jsplits > 1 ? (int)blockIdx.z * jper : 0, jend = min(nb, jbeg + jper);
  for (int j0 = jbeg; j0 < jend; j0 += TB) {
    float acc[8][QN];
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
      for (int q = 0; q < QN; ++q) acc[k][q] = 0.f;

    for (int c0 = 0; c0 < d; c0 += L1_DC) {
      __syncthreads();
      for (int idx = tid; idx < TA * 4; idx += nthr) {     // A chunk: TA rows x 4 pieces of 8 dims
        const int r = idx >> 2, c8 = (idx & 3) * 8, gi = i0 + r;
        float v[8];
        if (gi < na) l1_fetch8(pr.A, pr.a_f32, (long long)b * pr.sA + (long long)gi * d, c0 + c8, d, vec, v);
        else {
#pragma unroll
          for (int q = 0; q < 8; ++q) v[q] = 0.f;
        }
        *reinterpret_cast<float4*>(As + r * L1_PITCH + c8) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(As + r * L1_PITCH + c8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
      }
      for (int idx = tid; idx < TB * 4; idx += nthr) {     // B chunk
        const int r = idx >> 2, c8 = (idx & 3) * 8, gj = j0 + r;
        float v[8];
        if (gj < nb) l1_fetch8(args.Bm, args.b_f32, (long long)b * args.sB + (long long)gj * d, c0 + c8, d, vec, v);
        else {
#pragma unroll
          for (int q = 0; q < 8; ++q) v[q] = 0.f;
        }
        // the landmark operand is stored negated: a - b becomes one packed add per two dims
        *reinterpret_cast<float4*>(Bs + r * L1_PITCH + c8) = make_float4(-v[0], -v[1], -v[2], -v[3]);
        *reinterpret_cast<float4*>(Bs + r * L1_PITCH + c8 + 4) = make_float4(-v[4], -v[5], -v[6], -v[7]);
      }
      __syncthreads();
#pragma unroll
      for (int c4 = 0; c4 < L1_DC; c4 += 4) {
        ulonglong2 a[8], nb[QN];
#pragma unroll
        for (int k = 0; k < 8; ++k) a[k] = *reinterpret_cast<const ulonglong2*>(As + (ti + TG * k) * L1_PITCH + c4);
#pragma unroll
        for (int q = 0; q < QN; ++q) nb[q] = *reinterpret_cast<const ulonglong2*>(Bs + (tj + LG * q) * L1_PITCH + c4);
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
          for (int q = 0; q < QN; ++q) {
            const f32x2 t0 = add2(a[k].x, nb[q].x), t1 = add2(a[k].y, nb[q].y);   // dims c4, c4+1 and c4+2, c4+3
            acc[k][q] += fabsf(lo32(t0));
            acc[k][q] += fabsf(hi32(t0));
            acc[k][q] += fabsf(lo32(t1));
            acc[k][q] += fabsf(hi32(t1));
          }
      }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int gi = i0 + ti + TG * k;
      if (gi >= na) continue;
#pragma unroll
      for (int q = 0; q < QN; ++q) {
        const int gj = j0 + tj + LG * q;
        if (gj < nb) {
          const float e = ex2(acc[k][q] * args.nscale);
          E[(long long)gi * lde + gj] = e;
          rs[k] += e;
        } else if (gj < lde) {
          E[(long long)gi * lde + gj] = 0.f;   // padding columns of a padded leading dimension
        }
      }
    }
    if (pr.stat) {
      // Column statistics of this tile for the whitening scale (Eq. 5): per landmark the sums of t = E - pivot and of
      // t^2 over the tile's tokens, the pivot being the tile's first row (it makes t small, so that fp32 loses
      // nothing), moved to sums about zero in double by the thread that adds up the TG token groups in a fixed order.
      __syncthreads();                                   // every thread has finished reading the staged operands
      float* Ps = l1_smem;                               // [TB] pivots
      float* Sr = l1_smem + TB;                          // [TG][TB][2]
      if (ti == 0)
#pragma unroll
        for (int q = 0; q < QN; ++q) Ps[tj + LG * q] = ex2(acc[0][q] * args.nscale);
      __syncthreads();
#pragma unroll
      for (int q = 0; q < QN; ++q) {
        const float pv = Ps[tj + LG * q];
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (i0 + ti + TG * k < na) { const float t = ex2(acc[k][q] * args.nscale) - pv; s1 += t; s2 = fmaf(t, t, s2); }
        Sr[(ti * TB + tj + LG * q) * 2] = s1;
        Sr[(ti * TB + tj + LG * q) * 2 + 1] = s2;
      }
      __syncthreads();
      for (int c = tid; c < TB; c += nthr) {
        const int gj = j0 + c;
        if (gj < nb) {
          float a = 0.f, q2 = 0.f;
          for (int t = 0; t < TG; ++t) { a += Sr[(t * TB + c) * 2]; q2 += Sr[(t * TB + c) * 2 + 1]; }
          const double pv = (double)Ps[c], cnt = (double)min(TA, na - i0);
          double* o = pr.stat + (((long long)b * gridDim.x + blockIdx.x) * nb + gj) * 2;
          o[0] = (double)a + cnt * pv;
          o[1] = (double)q2 + 2.0 * pv * (double)a + cnt * pv * pv;
        }
      }
      __syncthreads();                                   // the staging buffers are free again for the next landmark tile
    }
  }
  if (pr.rowsum) {      // fixed-order reduction over the LG threads of a row
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; ++k) Rs[(ti + TG * k) * LG + tj] = rs[k];
    __syncthreads();
    for (int r = tid; r < TA; r += nthr) {
      float v = 0.f;
      for (int t = 0; t < LG; ++t) v += Rs[r * LG + t];
      if (i0 + r < na) pr.rowsum[(long long)b * na + i0 + r] = v * pr.rs_scale;
    }
  }
}

// =====================================================================================
// Whitening statistics (Eq. 5-6): per head h and landmark l, over the query rows of every batch element,
//     mu_l = mean C_il,  sigma_l^2 = mean (C_il - mu_l)^2,  s_l = 1 / sqrt(sigma_l^2 + eps).
// k_wstat_part: grid (splits, BH), block 256 = 64 column quads x 4 row lanes.  A thread walks its rows of its four
// columns sixteen at a time (four loads in flight): within the sixteen it adds t = C - pivot and t^2 in fp32 (the
// pivot, row 0 of the head, makes t small, so sixteen terms lose nothing), then adds the two short sums to double
// accumulators.  The four row lanes are added in a fixed order, the sums are moved from the pivot to zero in double,
// and the split leaves [m][2] doubles.  k_wstat_final adds the partial sums of all batch elements and splits in a
// fixed order and writes s.
// =====================================================================================
__global__ void __launch_bounds__(256) k_wstat_part(const float* __restrict__ C, int ldc, int n, int m, int rows_per_split,
                                                    double* __restrict__ part /* [BH][splits][m][2] */) {
  __shared__ double red[4][256][2];
  const int bh = blockIdx.y, split = blockIdx.x, nsplit = gridDim.x;
  const int cq = threadIdx.x & 63, rl = threadIdx.x >> 6, c0 = cq * 4;
  const float* Ch = C + (long long)bh * n * ldc;
  const int i0 = split * rows_per_split, i1 = min(n, i0 + rows_per_split);
  double s1[4] = {0.0, 0.0, 0.0, 0.0}, s2[4] = {0.0, 0.0, 0.0, 0.0};
  float4 pv = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c0 < ldc) {
    pv = *reinterpret_cast<const float4*>(Ch + c0);                 // pivot: row 0 of this head
    int i = i0 + rl;
    for (; i + 12 < i1; i += 16) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const float4*>(Ch + (long long)(i + 4 * u) * ldc + c0);
      float a[4] = {0.f, 0.f, 0.f, 0.f}, q[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float t0 = v[u].x - pv.x, t1 = v[u].y - pv.y, t2 = v[u].z - pv.z, t3 = v[u].w - pv.w;
        a[0] += t0; a[1] += t1; a[2] += t2; a[3] += t3;
        q[0] += t0 * t0; q[1] += t1 * t1; q[2] += t2 * t2; q[3] += t3 * t3;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) { s1[u] += (double)a[u]; s2[u] += (double)q[u]; }
    }
    for (; i < i1; i += 4) {
      const float4 v = *reinterpret_cast<const float4*>(Ch + (long long)i * ldc + c0);
      const float t0 = v.x - pv.x, t1 = v.y - pv.y, t2 = v.z - pv.z, t3 = v.w - pv.w;
      s1[0] += (double)t0; s1[1] += (double)t1; s1[2] += (double)t2; s1[3] += (double)t3;
      s2[0] += (double)(t0 * t0); s2[1] += (double)(t1 * t1); s2[2] += (double)(t2 * t2); s2[3] += (double)(t3 * t3);
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) { red[rl][cq * 4 + u][0] = s1[u]; red[rl][cq * 4 + u][1] = s2[u]; }
  __syncthreads();
  const int l = threadIdx.x;
  if (l < m) {
    const double a = (red[0][l][0] + red[1][l][0]) + (red[2][l][0] + red[3][l][0]);
    const double b = (red[0][l][1] + red[1][l][1]) + (red[2][l][1] + red[3][l][1]);
    // from sums about the pivot p to sums about zero: sum x = a + N p, sum x^2 = b + 2 p a + N p^2
    const double p = (double)Ch[l], cnt = (double)max(i1 - i0, 0);
    double* o = part + (((long long)bh * nsplit + split) * m + l) * 2;
    o[0] = a + cnt * p; o[1] = b + 2.0 * p * a + cnt * p * p;
  }
}

// grid (ceil(m / 32), H), block 256: lane = landmark of the group of 32, warp w adds terms w, w + 8, ... (term t = batch
// element t / nsplit, split t % nsplit; eight loads in flight), the eight warps are added in a fixed order
__global__ void __launch_bounds__(256) k_wstat_final(const double* __restrict__ part, int B, int H, int n, int m, int nsplit,
                                                     float eps, float* __restrict__ s_out /* [H][m] */,
                                                     float* __restrict__ mean_out /* NULL or [H][m] */) {
  __shared__ double red[8][32][2];
  const int h = blockIdx.y, lane = threadIdx.x & 31, w = threadIdx.x >> 5, l = blockIdx.x * 32 + lane;
  const int terms = B * nsplit;
  double sx = 0.0, sxx = 0.0;
  if (l < m) {
    int t = w, b = w / nsplit, sp = w % nsplit;
    auto next = [&](const double*& ptr) {               // address of term t, then on to term t + 8
      ptr = part + ((((long long)b * H + h) * nsplit + sp) * m + l) * 2;
      t += 8; sp += 8;
      while (sp >= nsplit) { sp -= nsplit; ++b; }
    };
    while (t + 56 < terms) {
      const double* q[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) next(q[u]);
      double2 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = *reinterpret_cast<const double2*>(q[u]);
#pragma unroll
      for (int u = 0; u < 8; ++u) { sx += v[u].x; sxx += v[u].y; }
    }
    while (t < terms) {
      const double* q; next(q);
      const double2 v = *reinterpret_cast<const double2*>(q);
      sx += v.x; sxx += v.y;
    }
  }
  red[w][lane][0] = sx; red[w][lane][1] = sxx;
  __syncthreads();
  if (w == 0 && l < m) {
    double a = 0.0, q = 0.0;
#pragma unroll
    for (int g = 0; g < 8; ++g) { a += red[g][lane][0]; q += red[g][lane][1]; }
    const double cnt = (double)B * (double)n;
    const double mu = a / cnt;
    double var = q / cnt - mu * mu;
    if (var < 0.0) var = 0.0;
    s_out[h * m + l] = (float)(1.0 / sqrt(var + (double)eps));
    if (mean_out) mean_out[h * m + l] = (float)mu;
  }
}

// Gradient of the loss with respect to the batch-statistic whitening scale, turned into the coefficient of the extra
// upstream term of the query-landmark block (Eq. 5-6 in training mode).  With Z_il = s_l (C_il - mu_i) + 1/m,
//     ds_l = sum_{b,i} (dO_i . Y_l)(C_il - mu_i) = sum_b <Y_l, ((C - mu)^T dO)_l>,
//     dsigma2_l = -1/2 s_l^3 ds_l,     dC_il += dsigma2_l (2/N)(C_il - cbar_l),   N = B n,
// so kap[h][l] = (kappa_l, cbar_l) with kappa_l = -s_l^3 ds_l / N.  One warp per (head, landmark): lanes run over the
// dims, batch elements and token chunks are added in a fixed order.  grid (ceil(m/8), H), block 256.
__global__ void __launch_bounds__(256) k_whiten_bwd(const float* __restrict__ Y, const float* __restrict__ dYtpart, int nchunks,
                                                    const float* __restrict__ s, const float* __restrict__ cbar, int B, int H,
                                                    int n, int m, int d, float* __restrict__ kap /* [H][m][2] */) {
  const int h = blockIdx.y, l = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (l >= m) return;
  float acc = 0.f;
  for (int b = 0; b < B; ++b) {
    const long long bh = (long long)b * H + h;
    for (int c = lane; c < d; c += 32) {
      float t = 0.f;
      for (int k = 0; k < nchunks; ++k) t += dYtpart[((bh * nchunks + k) * m + l) * d + c];
      acc = fmaf(Y[(bh * m + l) * d + c], t, acc);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const float sl = s[h * m + l];
    kap[(h * m + l) * 2] = -sl * sl * sl * acc / ((float)B * (float)n);
    kap[(h * m + l) * 2 + 1] = cbar[h * m + l];
  }
}

// G[i][l] += kappa_l (C[i][l] - cbar_l) C[i][l] / lambda: the extra upstream term of batch-statistic whitening for the
// paths that materialise G (fp32 storage, 32-dim heads).
__global__ void __launch_bounds__(256) k_g_whiten_add(float* __restrict__ G, const float* __restrict__ C, const float* __restrict__ kap,
                                                      int H, int n, int m, int ldm, float inv_lambda) {
  const int bh = blockIdx.y;
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
  if (e >= (long long)n * ldm) return;
  const int l = (int)(e % ldm);
  if (l >= m) return;
  const float* kp = kap + ((long long)(bh % H) * m + l) * 2;
  const long long idx = (long long)bh * n * ldm + e;
  const float c = C[idx];
  G[idx] += kp[0] * (c - kp[1]) * c * inv_lambda;
}

// storage type -> fp32 copy
template <typename T> __global__ void k_to_f32(const T* __restrict__ x, float* __restrict__ y, long long count) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) y[i] = to_f(x[i]);
}

// =====================================================================================
// Landmark selection: adaptive average pooling of the keys over the token grid (Sec. 4.2)
// =====================================================================================
// filt: NULL = average pooling; else the depth-wise-convolution selection of Sec. 4.2, one filter per head and channel,
// [H][taps][d] with taps = (gh/mh) * (gw/mw) (the grid divides: the host checks), tap (u, v) of a region at u (gw/mw) + v
struct PoolGeom { int n, d, m, prefix, gh, gw, mh, mw; const float* filt; int H; };
// 32-bit on purpose (64-bit division costs two orders of magnitude more on the device); the host
// checks that gh * mh and gw * mw stay below 2^31.
__host__ __device__ inline int bin_lo(int a, int g, int mb) { return (int)(((unsigned)a * (unsigned)g) / (unsigned)mb); }
__host__ __device__ inline int bin_hi(int a, int g, int mb) { return (int)(((unsigned)(a + 1) * (unsigned)g + (unsigned)mb - 1u) / (unsigned)mb); }

// grid (ceil(m / (256 / (d/4))), BH); thread = (landmark, 4 dims)
template <typename T>
__global__ void __launch_bounds__(256) k_pool(const T* __restrict__ K, float* __restrict__ L, PoolGeom g) {
  const int quads = g.d / 4, lpb = 256 / quads;
  const int l = blockIdx.x * lpb + (int)threadIdx.x / quads, bh = blockIdx.y, c = ((int)threadIdx.x % quads) * 4;
  if (l >= g.m || (int)threadIdx.x >= lpb * quads) return;
  const int a = l / g.mw, bb = l % g.mw;
  const int r0 = bin_lo(a, g.gh, g.mh), r1 = bin_hi(a, g.gh, g.mh);
  const int c0 = bin_lo(bb, g.gw, g.mw), c1 = bin_hi(bb, g.gw, g.mw);
  const T* Kh = K + (long long)bh * g.n * g.d;
  // The mean is accumulated in double and rounded once, so that the stored landmark is the fp32
  // value nearest to the exact mean: sign(token - landmark) in the backward pass then does not
  // depend on the order of a single-precision summation.
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  const float* wf = g.filt ? g.filt + (long long)(bh % g.H) * ((r1 - r0) * (c1 - c0)) * g.d + c : nullptr;
  for (int r = r0; r < r1; ++r)
    for (int q = c0; q < c1; ++q) {
      const float4 v = ld4(Kh + (long long)(g.prefix + r * g.gw + q) * g.d + c);
      if (wf) {                        // products of an fp32 weight and a token value are exact in double
        const float4 w = ld4(wf + (long long)((r - r0) * (c1 - c0) + (q - c0)) * g.d);
        s0 += (double)w.x * (double)v.x; s1 += (double)w.y * (double)v.y; s2 += (double)w.z * (double)v.z; s3 += (double)w.w * (double)v.w;
      } else { s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w; }
    }
  const double cnt = wf ? 1.0 : (double)((r1 - r0) * (c1 - c0));
  st4(L + ((long long)bh * g.m + l) * g.d + c,
      make_float4((float)(s0 / cnt), (float)(s1 / cnt), (float)(s2 / cnt), (float)(s3 / cnt)));
}

// The same for large bins (high-resolution grids): one CTA per (landmark, head), 256 threads = d/4 channel quads x
// 1024/d token lanes; lane t adds the bin's tokens t, t + lanes, ... in double (exact for any order at these sizes), the
// lanes are added in a fixed order.  With one thread per (landmark, quad) a 28 x 14 bin is a chain of 392 dependent loads.
template <typename T>
__global__ void __launch_bounds__(256) k_pool_wide(const T* __restrict__ K, float* __restrict__ L, PoolGeom g) {
  __shared__ double red[256][4];
  const int quads = g.d / 4, lanes = 256 / quads;
  const int l = blockIdx.x, bh = blockIdx.y, qd = (int)threadIdx.x % quads, tl = (int)threadIdx.x / quads, c = qd * 4;
  const int a = l / g.mw, bb = l % g.mw;
  const int r0 = bin_lo(a, g.gh, g.mh), r1 = bin_hi(a, g.gh, g.mh);
  const int c0 = bin_lo(bb, g.gw, g.mw), c1 = bin_hi(bb, g.gw, g.mw);
  const int bw = c1 - c0, cnt = (r1 - r0) * bw;
  const T* Kh = K + (long long)bh * g.n * g.d;
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  const float* wf = g.filt ? g.filt + (long long)(bh % g.H) * cnt * g.d + c : nullptr;
  if (tl < lanes)
    for (int t = tl; t < cnt; t += lanes) {
      const int r = r0 + t / bw, q = c0 + t % bw;
      const float4 v = ld4(Kh + (long long)(g.prefix + r * g.gw + q) * g.d + c);
      if (wf) {
        const float4 w = ld4(wf + (long long)t * g.d);
        s0 += (double)w.x * (double)v.x; s1 += (double)w.y * (double)v.y; s2 += (double)w.z * (double)v.z; s3 += (double)w.w * (double)v.w;
      } else { s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w; }
    }
  red[threadIdx.x][0] = s0; red[threadIdx.x][1] = s1; red[threadIdx.x][2] = s2; red[threadIdx.x][3] = s3;
  __syncthreads();
  if (tl == 0) {
    double t0 = 0.0, t1 = 0.0, t2 = 0.0, t3 = 0.0;
    for (int u = 0; u < lanes; ++u) { const double* p = red[u * quads + qd]; t0 += p[0]; t1 += p[1]; t2 += p[2]; t3 += p[3]; }
    const double n = wf ? 1.0 : (double)cnt;
    st4(L + ((long long)bh * g.m + l) * g.d + c, make_float4((float)(t0 / n), (float)(t1 / n), (float)(t2 / n), (float)(t3 / n)));
  }
}

// dK[j] = dKpart[j] (may be NULL) + sum over the bins containing token j of dL[bin] / |bin|
// (pooling adjoint); with pool == 0 it only converts dKpart to the storage type.
constexpr int POOL_EPT = 8;      // elements (of four dims) per thread of k_pool_bwd
template <typename T>
__global__ void __launch_bounds__(256, 4) k_pool_bwd(const float* __restrict__ dKpart, const float* __restrict__ dL, T* __restrict__ dK,
                                                  PoolGeom g, int pool) {
  // bin boundaries once per CTA (a division each) instead of several per thread
  __shared__ int rlo[256], rhi[256], clo[256], chi[256];
  __shared__ int s_lm[POOL_EPT * 256 / 8], s_tap[POOL_EPT * 256 / 8];   // per token of this CTA: its landmark and its tap (even bins)
  const int bh = blockIdx.y;
  const unsigned per_row = g.d / 4;
  const unsigned total = (unsigned)g.n * per_row;                  // n * d / 4 < 2^32
  const bool even = (g.gh % g.mh) == 0 && (g.gw % g.mw) == 0;      // the pooling of Sec. 4.2 proper: r x r windows, stride r
  const int bh_rows = g.gh / g.mh, bh_cols = g.gw / g.mw;
  const float even_inv = 1.f / (float)(bh_rows * bh_cols);
  // POOL_EPT elements of four dims per thread, a CTA's share contiguous, so that the tables are built once per 2048
  // elements.  With a head width of 32, 64 or 128 the share is 256, 128 or 64 whole tokens: their landmark (and tap) is
  // worked out once per token and CTA, and an element finds its token by a shift, not by five integer divisions.
  const bool table = pool && even && (per_row == 8u || per_row == 16u || per_row == 32u);
  const int sh = 31 - __clz((int)per_row);
  const unsigned base = blockIdx.x * (unsigned)(POOL_EPT * 256);
  const int j0 = (int)(base >> sh);
  // this CTA's share of the partial gradient is contiguous: one bulk copy (cp.async.bulk, up to 32 KB) stages it in
  // shared memory, so that the bytes in flight from HBM do not depend on the registers of the threads
  __shared__ __align__(128) float4 stage[POOL_EPT * 256];
  __shared__ __align__(8) unsigned long long bar;
  if (table && dKpart && threadIdx.x == 0) {
    const unsigned cnt = min(total - base, (unsigned)(POOL_EPT * 256));
    umma::mbar_init(&bar, 1);
    umma::mbar_expect_tx(&bar, cnt * 16u);
    umma::bulk_load(stage, dKpart + (long long)bh * g.n * g.d + (long long)base * 4, cnt * 16u, &bar);
  }
  if (pool) {
    if (!table) {
      for (int a = threadIdx.x; a < g.mh; a += 256) { rlo[a] = bin_lo(a, g.gh, g.mh); rhi[a] = bin_hi(a, g.gh, g.mh); }
      for (int b = threadIdx.x; b < g.mw; b += 256) { clo[b] = bin_lo(b, g.gw, g.mw); chi[b] = bin_hi(b, g.gw, g.mw); }
    } else {
      for (int t = threadIdx.x; t < ((POOL_EPT * 256) >> sh); t += 256) {
        const int j = j0 + t;
        int lm = -1, tap = 0;
        if (j < g.n && j >= g.prefix) {
          const int r = (j - g.prefix) / g.gw, q = (j - g.prefix) % g.gw;
          lm = (r / bh_rows) * g.mw + q / bh_cols;
          tap = (r % bh_rows) * bh_cols + q % bh_cols;
        }
        s_lm[t] = lm; s_tap[t] = tap;
      }
    }
    __syncthreads();
  }
  if (table) {
    // the landmark rows (L2) are loaded while the bulk copy of the partial gradient (HBM) is on its way
    float4 t[POOL_EPT];
    int lm[POOL_EPT];
#pragma unroll
    for (int u = 0; u < POOL_EPT; ++u) {
      const unsigned idx = base + (unsigned)u * 256u + threadIdx.x;
      lm[u] = idx < total ? s_lm[(int)(idx >> sh) - j0] : -2;    // -2: past the end; -1: a prefix token
      t[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lm[u] >= 0) t[u] = ld4(dL + ((long long)bh * g.m + lm[u]) * g.d + (int)(idx & (per_row - 1u)) * 4);
    }
    // a wait that ran out (it cannot, short of a fault elsewhere) falls back to plain loads of the same values
    const bool staged = dKpart != nullptr && umma::mbar_wait(&bar, 0);
#pragma unroll
    for (int u = 0; u < POOL_EPT; ++u) {
      if (lm[u] == -2) continue;
      const unsigned idx = base + (unsigned)u * 256u + threadIdx.x;
      float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
      if (staged) o = stage[u * 256 + threadIdx.x];
      else if (dKpart) o = ld4(dKpart + (long long)bh * g.n * g.d + (long long)idx * 4);
      if (lm[u] >= 0) {
        float4 w = make_float4(even_inv, even_inv, even_inv, even_inv);
        if (g.filt) w = ld4(g.filt + ((long long)(bh % g.H) * (bh_rows * bh_cols) + s_tap[(int)(idx >> sh) - j0]) * g.d + (int)(idx & (per_row - 1u)) * 4);
        o.x += t[u].x * w.x; o.y += t[u].y * w.y; o.z += t[u].z * w.z; o.w += t[u].w * w.w;
      }
      st4(dK + (long long)bh * g.n * g.d + (long long)idx * 4, o);
    }
    return;
  }
#pragma unroll
  for (int u = 0; u < POOL_EPT; ++u) {
    const unsigned idx = (blockIdx.x * POOL_EPT + u) * blockDim.x + threadIdx.x;
    if (idx >= total) break;
    const int j = (int)(idx / per_row), c = (int)(idx % per_row) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (dKpart) v = ld4(dKpart + ((long long)bh * g.n + j) * g.d + c);
    if (pool && j >= g.prefix && even) {
      // bins of equal size that do not overlap: one bin per token
      const int r = (j - g.prefix) / g.gw, q = (j - g.prefix) % g.gw;
      const float4 t = ld4(dL + ((long long)bh * g.m + (r / bh_rows) * g.mw + q / bh_cols) * g.d + c);
      if (g.filt) {                      // selection filter: the token's tap of its region
        const float4 w = ld4(g.filt + ((long long)(bh % g.H) * (bh_rows * bh_cols) + (r % bh_rows) * bh_cols + q % bh_cols) * g.d + c);
        v.x += t.x * w.x; v.y += t.y * w.y; v.z += t.z * w.z; v.w += t.w * w.w;
      } else { v.x += t.x * even_inv; v.y += t.y * even_inv; v.z += t.z * even_inv; v.w += t.w * even_inv; }
    } else if (pool && j >= g.prefix) {
      const int r = (j - g.prefix) / g.gw, q = (j - g.prefix) % g.gw;
      // a token row lies in bin floor(r mh / gh) and, where neighbouring bins overlap, in the next one too
      const int a0 = (int)(((unsigned)r * (unsigned)g.mh) / (unsigned)g.gh), b0 = (int)(((unsigned)q * (unsigned)g.mw) / (unsigned)g.gw);
      for (int a = (a0 > 0 ? a0 - 1 : 0); a <= a0 + 1 && a < g.mh; ++a) {
        if (r < rlo[a] || r >= rhi[a]) continue;
        for (int bb = (b0 > 0 ? b0 - 1 : 0); bb <= b0 + 1 && bb < g.mw; ++bb) {
          if (q < clo[bb] || q >= chi[bb]) continue;
          const float inv = 1.f / (float)((rhi[a] - rlo[a]) * (chi[bb] - clo[bb]));
          const float4 t = ld4(dL + ((long long)bh * g.m + a * g.mw + bb) * g.d + c);
          v.x += t.x * inv; v.y += t.y * inv; v.z += t.z * inv; v.w += t.w * inv;
        }
      }
    }
    st4(dK + ((long long)bh * g.n + j) * g.d + c, v);
  }
}

// The same for many parts (one per token tile of the sign passes): warp w of a CTA adds the parts w, w + 8, ... of every
// array for 128 consecutive elements (four loads in flight per thread), the eight warps are added in a fixed order.
// Eight times the CTAs of k_reduce3, which on long sequences has too few of them to draw the memory bandwidth.
__device__ __forceinline__ float4 sum_parts4_strided(const float* __restrict__ parts, int nparts, long long stride, long long off, int first, int step) {
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  int p = first;
  for (; p + 3 * step < nparts; p += 4 * step) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const float4*>(parts + (long long)(p + u * step) * stride + off);
#pragma unroll
    for (int u = 0; u < 4; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
  }
  for (; p < nparts; p += step) {
    const float4 v = *reinterpret_cast<const float4*>(parts + (long long)p * stride + off);
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  return s;
}
template <typename TO>
__global__ void __launch_bounds__(256) k_reduce3_wide(const float* __restrict__ p0, int n0, const float* __restrict__ p1, int n1,
                                                      const float* __restrict__ p2, int n2, TO* __restrict__ out, int count) {
  __shared__ float4 red[8][32];
  const int bh = blockIdx.y, w = threadIdx.x >> 5, l = threadIdx.x & 31;
  const int e = (blockIdx.x * 32 + l) * 4;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (e < count) {
    s = sum_parts4_strided(p0 + (long long)bh * n0 * count, n0, count, e, w, 8);
    if (n1 > 0) { const float4 t = sum_parts4_strided(p1 + (long long)bh * n1 * count, n1, count, e, w, 8); s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w; }
    if (n2 > 0) { const float4 t = sum_parts4_strided(p2 + (long long)bh * n2 * count, n2, count, e, w, 8); s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w; }
  }
  red[w][l] = s;
  __syncthreads();
  if (w == 0 && e < count) {
    float4 t = red[0][l];
#pragma unroll
    for (int k = 1; k < 8; ++k) { t.x += red[k][l].x; t.y += red[k][l].y; t.z += red[k][l].z; t.w += red[k][l].w; }
    st4(out + (long long)bh * count + e, t);
  }
}

// Gradient of the landmark-selection filter: dF[h][tap][c] = sum over the batch elements b and the landmarks l of
// dL[b H + h][l][c] X[b H + h][token(l, tap)][c], X the tensor the landmarks were selected from.
// grid (taps, H, splits); 256 threads = d/4 channel quads x 1024/d lanes over the (b, l) pairs of this split; double sums,
// lanes added in order.  With splits > 1 the CTAs write partial sums [split][H][taps][d] that k_filter_reduce adds up in a
// fixed order (taps x H alone are too few CTAs where the batch is large).
template <typename T>
__global__ void __launch_bounds__(256) k_filter_grad(const T* __restrict__ X, const float* __restrict__ dL, float* __restrict__ dF,
                                                     PoolGeom g, int B) {
  __shared__ double red[256][4];
  const int quads = g.d / 4, lanes = 256 / quads;
  const int tap = blockIdx.x, h = blockIdx.y, qd = (int)threadIdx.x % quads, tl = (int)threadIdx.x / quads, c = qd * 4;
  const int rh = g.gh / g.mh, rw = g.gw / g.mw, u = tap / rw, v = tap % rw;
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
  const int pairs = B * g.m, per = (pairs + (int)gridDim.z - 1) / (int)gridDim.z;
  const int t_beg = (int)blockIdx.z * per, t_end = min(pairs, t_beg + per);
  if (tl < lanes) {
    auto addr = [&](int t, const T*& xp, const float*& lp) {
      const int b = t / g.m, l = t % g.m, a = l / g.mw, bb = l % g.mw;
      const long long bh = (long long)b * g.H + h;
      xp = X + (bh * g.n + g.prefix + (a * rh + u) * g.gw + (bb * rw + v)) * g.d + c;
      lp = dL + (bh * g.m + l) * g.d + c;
    };
    int t = t_beg + tl;
    for (; t + 3 * lanes < t_end; t += 4 * lanes) {        // four pairs in flight per thread
      float4 x[4], dl[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const T* xp; const float* lp;
        addr(t + q * lanes, xp, lp);
        x[q] = ld4(xp); dl[q] = ld4(lp);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        s0 += (double)dl[q].x * (double)x[q].x; s1 += (double)dl[q].y * (double)x[q].y;
        s2 += (double)dl[q].z * (double)x[q].z; s3 += (double)dl[q].w * (double)x[q].w;
      }
    }
    for (; t < t_end; t += lanes) {
      const T* xp; const float* lp;
      addr(t, xp, lp);
      const float4 x = ld4(xp), dl = ld4(lp);
      s0 += (double)dl.x * (double)x.x; s1 += (double)dl.y * (double)x.y; s2 += (double)dl.z * (double)x.z; s3 += (double)dl.w * (double)x.w;
    }
  }
  red[threadIdx.x][0] = s0; red[threadIdx.x][1] = s1; red[threadIdx.x][2] = s2; red[threadIdx.x][3] = s3;
  __syncthreads();
  if (tl == 0) {
    double t0 = 0.0, t1 = 0.0, t2 = 0.0, t3 = 0.0;
    for (int w = 0; w < lanes; ++w) { const double* p = red[w * quads + qd]; t0 += p[0]; t1 += p[1]; t2 += p[2]; t3 += p[3]; }
    st4(dF + (((long long)blockIdx.z * g.H + h) * (rh * rw) + tap) * g.d + c, make_float4((float)t0, (float)t1, (float)t2, (float)t3));
  }
}
// dF[e] = sum over the splits of part[split][e], in order; count = H taps d (a multiple of 4)
__global__ void __launch_bounds__(256) k_filter_reduce(const float* __restrict__ part, int splits, float* __restrict__ dF, int count) {
  const int e = (blockIdx.x * 256 + threadIdx.x) * 4;
  if (e >= count) return;
  st4(dF + e, sum_parts4(part, splits, count, e));
}

// out[e] = sum_p parts[p][e] for up to three part arrays laid out [BH][np][count]; count % 4 == 0
template <typename TO>
__global__ void k_reduce3(const float* __restrict__ p0, int n0, const float* __restrict__ p1, int n1,
                          const float* __restrict__ p2, int n2, TO* __restrict__ out, int count) {
  const int bh = blockIdx.y;
  const int e = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (e >= count) return;
  float4 s = sum_parts4(p0 + (long long)bh * n0 * count, n0, count, e);
  if (n1 > 0) { const float4 t = sum_parts4(p1 + (long long)bh * n1 * count, n1, count, e); s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w; }
  if (n2 > 0) { const float4 t = sum_parts4(p2 + (long long)bh * n2 * count, n2, count, e); s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w; }
  st4(out + (long long)bh * count + e, s);
}

// =====================================================================================
// part[chunk][l][c] = sum_{j in chunk} (E[j][l] - mu[j]) * U[j][c]     (reduction over tokens)
// Used for M = R V (mu = NULL) and for the centred Z'^T dO of the backward pass.
// Optionally also colsum_part[chunk][c] = sum_j U[j][c].
// grid (chunks, ceil(m/64), BH); thread: 4 landmarks x D/16 columns
// =====================================================================================
template <typename TU, int D>
__global__ void __launch_bounds__(256) k_tn(const float* __restrict__ E, int lde, const float* __restrict__ mu,
                                            const TU* __restrict__ U, float* __restrict__ part,
                                            float* __restrict__ colsum_part, int n, int m, int rpc) {
  constexpr int DC = D / 16;
  __shared__ __align__(16) float Es[32][64 + 4];
  __shared__ __align__(16) float Us[32][D + 4];
  const int chunk = blockIdx.x, l0 = blockIdx.y * 64, bh = blockIdx.z, nchunks = gridDim.x;
  const int tid = threadIdx.x, tl = tid >> 4, tc = tid & 15;
  E += (long long)bh * n * lde;
  U += (long long)bh * n * D;
  if (mu) mu += (long long)bh * n;
  const int jbeg = chunk * rpc, jend = min(n, jbeg + rpc);
  float acc[4][DC], cs[DC];
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int q = 0; q < DC; ++q) acc[k][q] = 0.f;
#pragma unroll
  for (int q = 0; q < DC; ++q) cs[q] = 0.f;

  for (int j0 = jbeg; j0 < jend; j0 += 32) {
    __syncthreads();
    {  // E tile: 32 tokens x 64 landmarks, 8 per thread
      const int r = tid >> 3, cb = (tid & 7) * 8, j = j0 + r;
      const float mj = (mu && j < jend) ? mu[j] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 4) {
        const int l = l0 + cb + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < jend && l < m) {
          if (l + 3 < lde && (lde & 3) == 0) v = ld4(E + (long long)j * lde + l);
          else {
            v.x = E[(long long)j * lde + l];
            if (l + 1 < m) v.y = E[(long long)j * lde + l + 1];
            if (l + 2 < m) v.z = E[(long long)j * lde + l + 2];
            if (l + 3 < m) v.w = E[(long long)j * lde + l + 3];
          }
          v.x = (l < m) ? v.x - mj : 0.f;
          v.y = (l + 1 < m) ? v.y - mj : 0.f;
          v.z = (l + 2 < m) ? v.z - mj : 0.f;
          v.w = (l + 3 < m) ? v.w - mj : 0.f;
        }
        *reinterpret_cast<float4*>(&Es[r][cb + k]) = v;
      }
    }
    for (int idx = tid; idx < 32 * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4, j = j0 + r;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (j < jend) v = ld4(U + (long long)j * D + c4);
      *reinterpret_cast<float4*>(&Us[r][c4]) = v;
    }
    __syncthreads();
#pragma unroll 4
    for (int jj = 0; jj < 32; ++jj) {
      const float4 e4 = *reinterpret_cast<const float4*>(&Es[jj][tl * 4]);
      float u[DC];
      ld_cols<D>(&Us[jj][0], tc, u);
      const float e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int q = 0; q < DC; ++q) acc[k][q] = fmaf(e[k], u[q], acc[k][q]);
      if (colsum_part && tl == 0)
#pragma unroll
        for (int q = 0; q < DC; ++q) cs[q] += u[q];
    }
  }
  float* out = part + ((long long)bh * nchunks + chunk) * m * D;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int l = l0 + tl * 4 + k;
    if (l < m)
#pragma unroll
      for (int q = 0; q < DC; ++q) out[(long long)l * D + ColMap<D>::col(tc, q)] = acc[k][q];
  }
  if (colsum_part && tl == 0 && blockIdx.y == 0)
#pragma unroll
    for (int q = 0; q < DC; ++q) colsum_part[((long long)bh * nchunks + chunk) * D + ColMap<D>::col(tc, q)] = cs[q];
}

// =====================================================================================
// O[i][c] = sum_l (E[i][l] - mu[i]) * Y[l][c] + ybar[c]      (reduction over landmarks)
// Used for O = Z' Ytilde + ybar (Eq. 7 in folded form) and dV = R^T dM (mu, ybar = NULL).
// grid (ceil(n/64), BH); thread: 4 tokens x D/16 columns
// =====================================================================================
template <typename TO, int D>
__global__ void __launch_bounds__(256) k_nn(const float* __restrict__ E, int lde, const float* __restrict__ mu,
                                            const float* __restrict__ Y, const float* __restrict__ ybar,
                                            TO* __restrict__ O, int n, int m) {
  constexpr int DC = D / 16;
  __shared__ __align__(16) float Es[64][32 + 4];
  __shared__ __align__(16) float Ys[32][D + 4];
  const int i0 = blockIdx.x * 64, bh = blockIdx.y;
  const int tid = threadIdx.x, tt = tid >> 4, tc = tid & 15;
  E += (long long)bh * n * lde;
  Y += (long long)bh * m * D;
  O += (long long)bh * n * D;
  float acc[4][DC];
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int q = 0; q < DC; ++q) acc[k][q] = 0.f;

  for (int l0 = 0; l0 < m; l0 += 32) {
    __syncthreads();
    {  // E tile: 64 tokens x 32 landmarks
      const int r = tid >> 2, cb = (tid & 3) * 8, i = i0 + r;
      const float mi = (mu && i < n) ? mu[(long long)bh * n + i] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 4) {
        const int l = l0 + cb + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < n && l < m) {
          if (l + 3 < lde && (lde & 3) == 0) v = ld4(E + (long long)i * lde + l);
          else {
            v.x = E[(long long)i * lde + l];
            if (l + 1 < m) v.y = E[(long long)i * lde + l + 1];
            if (l + 2 < m) v.z = E[(long long)i * lde + l + 2];
            if (l + 3 < m) v.w = E[(long long)i * lde + l + 3];
          }
          v.x = (l < m) ? v.x - mi : 0.f;
          v.y = (l + 1 < m) ? v.y - mi : 0.f;
          v.z = (l + 2 < m) ? v.z - mi : 0.f;
          v.w = (l + 3 < m) ? v.w - mi : 0.f;
        }
        *reinterpret_cast<float4*>(&Es[r][cb + k]) = v;
      }
    }
    for (int idx = tid; idx < 32 * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4, l = l0 + r;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l < m) v = ld4(Y + (long long)l * D + c4);
      *reinterpret_cast<float4*>(&Ys[r][c4]) = v;
    }
    __syncthreads();
#pragma unroll 2
    for (int ll = 0; ll < 32; ll += 4) {
      float e[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 t = *reinterpret_cast<const float4*>(&Es[tt * 4 + k][ll]);
        e[k][0] = t.x; e[k][1] = t.y; e[k][2] = t.z; e[k][3] = t.w;
      }
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        float y[DC];
        ld_cols<D>(&Ys[ll + s][0], tc, y);
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
          for (int q = 0; q < DC; ++q) acc[k][q] = fmaf(e[k][s], y[q], acc[k][q]);
      }
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = i0 + tt * 4 + k;
    if (i < n)
#pragma unroll
      for (int q = 0; q < DC; ++q) {
        const int c = ColMap<D>::col(tc, q);
        const float yb = ybar ? ybar[(long long)bh * D + c] : 0.f;
        O[(long long)i * D + c] = from_f<TO>(acc[k][q] + yb);
      }
  }
}

// =====================================================================================
// G[i][l] = (sum_c U[i][c] * Y[l][c]) * E[i][l] / lambda       (reduction over d)
// The upstream gradient of a kernel block times the kernel value (App. A): with U = dO, Y = Ytilde
// it is dC o C / lambda, with U = V, Y = dM it is dR o R / lambda.
// grid (ceil(n/64), ceil(m/64), BH); thread: tokens tt*4+k, landmarks tl+16q
// =====================================================================================
template <typename TU, int D>
__global__ void __launch_bounds__(256) k_nt_g(const TU* __restrict__ U, const float* __restrict__ Y,
                                              const float* __restrict__ E, int lde, float* __restrict__ G,
                                              int n, int m, float inv_lambda) {
  constexpr int DK = (D < 64) ? D : 64;
  __shared__ __align__(16) float Us[64][DK + 4];
  __shared__ __align__(16) float Ys[64][DK + 4];
  const int i0 = blockIdx.x * 64, l0 = blockIdx.y * 64, bh = blockIdx.z;
  const int tid = threadIdx.x, tt = tid >> 4, tl = tid & 15;
  U += (long long)bh * n * D;
  Y += (long long)bh * m * D;
  E += (long long)bh * n * lde;
  G += (long long)bh * n * lde;
  float acc[4][4];
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[k][q] = 0.f;
  for (int c0 = 0; c0 < D; c0 += DK) {
    __syncthreads();
    for (int idx = tid; idx < 64 * (DK / 4); idx += 256) {
      const int r = idx / (DK / 4), c4 = (idx % (DK / 4)) * 4;
      float4 u = make_float4(0.f, 0.f, 0.f, 0.f), y = u;
      if (i0 + r < n) u = ld4(U + (long long)(i0 + r) * D + c0 + c4);
      if (l0 + r < m) y = ld4(Y + (long long)(l0 + r) * D + c0 + c4);
      *reinterpret_cast<float4*>(&Us[r][c4]) = u;
      *reinterpret_cast<float4*>(&Ys[r][c4]) = y;
    }
    __syncthreads();
#pragma unroll 4
    for (int c = 0; c < DK; c += 4) {
      float4 u[4], y[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) u[k] = *reinterpret_cast<const float4*>(&Us[tt * 4 + k][c]);
#pragma unroll
      for (int q = 0; q < 4; ++q) y[q] = *reinterpret_cast<const float4*>(&Ys[tl + 16 * q][c]);
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int q = 0; q < 4; ++q)
          acc[k][q] += u[k].x * y[q].x + u[k].y * y[q].y + u[k].z * y[q].z + u[k].w * y[q].w;
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = i0 + tt * 4 + k;
    if (i >= n) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int l = l0 + tl + 16 * q;
      if (l < m) G[(long long)i * lde + l] = acc[k][q] * E[(long long)i * lde + l] * inv_lambda;
      else if (l < lde) G[(long long)i * lde + l] = 0.f;
    }
  }
}

// =====================================================================================
// Sign pass over the landmarks (App. A):  out[i][c] = -sum_l G[i][l] * sign(tok[i][c] - L[l][c])
// grid (ceil(n/64), BH[, splits]); thread: 4 tokens x D/16 dims, token values held in registers.
// lper > 0 (a multiple of 32): blockIdx.z takes the landmarks [z lper, (z + 1) lper) and writes the partial sum
// out[bh][z][n][D] (few, long rows of landmarks: the stand-alone kernel gradient).  Gk != NULL: the factor is formed on
// the fly as G[i][l] Gk[i][l] gscale (upstream gradient times kernel value over lambda).
template <typename TT, typename TL, typename TO, int D>
__global__ void __launch_bounds__(256) k_sign_rows(const TT* __restrict__ tok, const TL* __restrict__ Lm,
                                                   const float* __restrict__ G, int ldg, TO* __restrict__ out,
                                                   int n, int m, int lper = 0, const float* __restrict__ Gk = nullptr,
                                                   float gscale = 1.f) {
  constexpr int DC = D / 16;
  __shared__ __align__(16) float Ls[32][D + 4];
  __shared__ __align__(16) float Gs[64][32 + 4];
  const int i0 = blockIdx.x * 64, bh = blockIdx.y;
  const int tid = threadIdx.x, tt = tid >> 4, tc = tid & 15;
  tok += (long long)bh * n * D;
  Lm += (long long)bh * m * D;
  G += (long long)bh * n * ldg;
  if (Gk) Gk += (long long)bh * n * ldg;
  const int lbeg = lper > 0 ? (int)blockIdx.z * lper : 0, lend = lper > 0 ? min(m, lbeg + lper) : m;
  out += lper > 0 ? ((long long)bh * gridDim.z + blockIdx.z) * n * D : (long long)bh * n * D;
  constexpr int DP = DC / 2;                 // packed pairs of adjacent dims
  f32x2 qp[4][DP], acc[4][DP];
  float gsum[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = i0 + tt * 4 + k;
    gsum[k] = 0.f;
#pragma unroll
    for (int s = 0; s < DP; ++s) {
      acc[k][s] = 0ull;
      const float q0 = (i < n) ? to_f(tok[(long long)i * D + ColMap<D>::col(tc, 2 * s)]) : 0.f;
      const float q1 = (i < n) ? to_f(tok[(long long)i * D + ColMap<D>::col(tc, 2 * s + 1)]) : 0.f;
      qp[k][s] = pack2(q0, q1);
    }
  }
  for (int l0 = lbeg; l0 < lend; l0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l0 + r < lend) v = ld4(Lm + (long long)(l0 + r) * D + c4);
      *reinterpret_cast<float4*>(&Ls[r][c4]) = make_float4(-v.x, -v.y, -v.z, -v.w);   // negated: q - L is a packed add
    }
    {  // G tile: 64 tokens x 32 landmarks (zero outside)
      const int r = tid >> 2, cb = (tid & 3) * 8, i = i0 + r;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int l = l0 + cb + k;
        float gv = (i < n && l < lend) ? G[(long long)i * ldg + l] : 0.f;
        if (Gk && i < n && l < lend) gv *= Gk[(long long)i * ldg + l] * gscale;
        Gs[r][cb + k] = gv;
      }
    }
    __syncthreads();
    const int lcount = min(32, (lend - l0 + 3) & ~3);  // landmarks of this chunk, rounded up to 4 (the rest is zero)
#pragma unroll 2
    for (int ll = 0; ll < lcount; ll += 4) {
      float g[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 t = *reinterpret_cast<const float4*>(&Gs[tt * 4 + k][ll]);
        g[k][0] = t.x; g[k][1] = t.y; g[k][2] = t.z; g[k][3] = t.w;
      }
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        f32x2 nl[DP];
        ld_col_pairs<D>(&Ls[ll + s][0], tc, nl);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          gsum[k] += g[k][s];
          const f32x2 gg = pack2(g[k][s], g[k][s]);
#pragma unroll
          for (int c = 0; c < DP; ++c) acc[k][c] = sign_step2(qp[k][c], nl[c], gg, acc[k][c]);
        }
      }
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = i0 + tt * 4 + k;
    if (i < n)
#pragma unroll
      for (int c = 0; c < DP; ++c) {
        out[(long long)i * D + ColMap<D>::col(tc, 2 * c)] = from_f<TO>(gsum[k] - 2.f * lo32(acc[k][c]));
        out[(long long)i * D + ColMap<D>::col(tc, 2 * c + 1)] = from_f<TO>(gsum[k] - 2.f * hi32(acc[k][c]));
      }
  }
}

// =====================================================================================
// Sign pass over the tokens:  part[chunk][l][c] = +sum_{i in chunk} G[i][l] * sign(tok[i][c] - L[l][c])
// grid (chunks, ceil(m/64), BH); thread: 4 landmarks x D/16 dims, landmark values in registers
// =====================================================================================
template <typename TT, typename TL, int D>
__global__ void __launch_bounds__(256) k_sign_cols(const TT* __restrict__ tok, const TL* __restrict__ Lm,
                                                   const float* __restrict__ G, int ldg, float* __restrict__ part,
                                                   int n, int m, int rpc, const float* __restrict__ Gk = nullptr,
                                                   float gscale = 1.f) {
  constexpr int DC = D / 16;
  __shared__ __align__(16) float Ts[32][D + 4];
  __shared__ __align__(16) float Gs[32][64 + 4];
  const int chunk = blockIdx.x, l0 = blockIdx.y * 64, bh = blockIdx.z, nchunks = gridDim.x;
  const int tid = threadIdx.x, tl = tid >> 4, tc = tid & 15;
  tok += (long long)bh * n * D;
  Lm += (long long)bh * m * D;
  G += (long long)bh * n * ldg;
  if (Gk) Gk += (long long)bh * n * ldg;
  const int ibeg = chunk * rpc, iend = min(n, ibeg + rpc);
  constexpr int DP = DC / 2;
  f32x2 nl[4][DP], acc[4][DP];                // negated landmark values, accumulators, as pairs of adjacent dims
  float gsum[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int l = l0 + tl * 4 + k;
    gsum[k] = 0.f;
#pragma unroll
    for (int s = 0; s < DP; ++s) {
      acc[k][s] = 0ull;
      const float v0 = (l < m) ? to_f(Lm[(long long)l * D + ColMap<D>::col(tc, 2 * s)]) : 0.f;
      const float v1 = (l < m) ? to_f(Lm[(long long)l * D + ColMap<D>::col(tc, 2 * s + 1)]) : 0.f;
      nl[k][s] = pack2(-v0, -v1);
    }
  }
  for (int j0 = ibeg; j0 < iend; j0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (j0 + r < iend) v = ld4(tok + (long long)(j0 + r) * D + c4);
      *reinterpret_cast<float4*>(&Ts[r][c4]) = v;
    }
    {  // G tile: 32 tokens x 64 landmarks (zero outside)
      const int r = tid >> 3, cb = (tid & 7) * 8, i = j0 + r;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int l = l0 + cb + k;
        float gv = (i < iend && l < m) ? G[(long long)i * ldg + l] : 0.f;
        if (Gk && i < iend && l < m) gv *= Gk[(long long)i * ldg + l] * gscale;
        Gs[r][cb + k] = gv;
      }
    }
    __syncthreads();
    const int jcount = min(32, iend - j0);
#pragma unroll 4
    for (int jj = 0; jj < jcount; ++jj) {
      const float4 g4 = *reinterpret_cast<const float4*>(&Gs[jj][tl * 4]);
      const float g[4] = {g4.x, g4.y, g4.z, g4.w};
      f32x2 tv[DP];
      ld_col_pairs<D>(&Ts[jj][0], tc, tv);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        gsum[k] += g[k];
        const f32x2 gg = pack2(g[k], g[k]);
#pragma unroll
        for (int c = 0; c < DP; ++c) acc[k][c] = sign_step2(tv[c], nl[k][c], gg, acc[k][c]);
      }
    }
  }
  float* out = part + ((long long)bh * nchunks + chunk) * m * D;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int l = l0 + tl * 4 + k;
    if (l < m)
#pragma unroll
      for (int c = 0; c < DP; ++c) {
        out[(long long)l * D + ColMap<D>::col(tc, 2 * c)] = 2.f * lo32(acc[k][c]) - gsum[k];
        out[(long long)l * D + ColMap<D>::col(tc, 2 * c + 1)] = 2.f * hi32(acc[k][c]) - gsum[k];
      }
  }
}

// =====================================================================================
// Whole-CTA fp32 GEMM on global (L2-resident) row-major matrices:
//   C = beta * Cin + alpha * op(A) op(B),  op(A) is M x K, op(B) is K x N.
// Executed by all 256 threads of a CTA; ends with __syncthreads(), so a following call may
// read C.  Cin may equal C (each element is read and written by the same thread).
// =====================================================================================
struct GemmSmem { float As[16][64 + 4]; float Bs[16][64 + 4]; };

template <bool TRA, bool TRB>
__device__ void cta_gemm(int M, int N, int K, const float* A, int lda, const float* Bm, int ldb,
                         float* C, int ldc, float alpha, float beta, const float* Cin, GemmSmem& sm, int part = 0, int nparts = 1) {
  // nparts CTAs of a cluster share the product: output tile t goes to CTA t % nparts
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  int tile = 0;
  for (int i0 = 0; i0 < M; i0 += 64)
    for (int j0 = 0; j0 < N; j0 += 64) {
      if ((tile++) % nparts != part) continue;
      float acc[4][4];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int s = 0; s < 4; ++s) acc[r][s] = 0.f;
      for (int k0 = 0; k0 < K; k0 += 16) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int idx = tid + e * 256;   // 1024 elements per operand tile
          if (TRA) {                       // op(A)(i,k) = A[k][i]: i fastest
            const int kk = idx >> 6, i = idx & 63;
            sm.As[kk][i] = (k0 + kk < K && i0 + i < M) ? A[(long long)(k0 + kk) * lda + i0 + i] : 0.f;
          } else {                         // op(A)(i,k) = A[i][k]: k fastest
            const int i = idx >> 4, kk = idx & 15;
            sm.As[kk][i] = (k0 + kk < K && i0 + i < M) ? A[(long long)(i0 + i) * lda + k0 + kk] : 0.f;
          }
          if (TRB) {                       // op(B)(k,j) = B[j][k]: k fastest
            const int j = idx >> 4, kk = idx & 15;
            sm.Bs[kk][j] = (k0 + kk < K && j0 + j < N) ? Bm[(long long)(j0 + j) * ldb + k0 + kk] : 0.f;
          } else {                         // op(B)(k,j) = B[k][j]: j fastest
            const int kk = idx >> 6, j = idx & 63;
            sm.Bs[kk][j] = (k0 + kk < K && j0 + j < N) ? Bm[(long long)(k0 + kk) * ldb + j0 + j] : 0.f;
          }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
          const float4 a = *reinterpret_cast<const float4*>(&sm.As[kk][ty * 4]);
          const float4 b = *reinterpret_cast<const float4*>(&sm.Bs[kk][tx * 4]);
          const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int s = 0; s < 4; ++s) acc[r][s] = fmaf(av[r], bv[s], acc[r][s]);
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = i0 + ty * 4 + r;
        if (i >= M) continue;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const int j = j0 + tx * 4 + s;
          if (j >= N) continue;
          float v = alpha * acc[r][s];
          if (beta != 0.f) v += beta * Cin[(long long)i * ldc + j];
          C[(long long)i * ldc + j] = v;
        }
      }
    }
  __syncthreads();
}

// Shared memory of the per-head kernels: one of the two GEMM engines is used per instantiation.
union __align__(16) NsSmem { GemmSmem f; MmaGemmSmem t; };

// C = beta*Cin + alpha*op(A)op(B) + diag*I on either engine: TC = tensor cores with split-bf16
// operands (bf16-storage path), else exact fp32 FFMA (fp32-storage path, stand-alone ns_pinv).
template <bool TC, bool TRA, bool TRB, bool BIG = false>
__device__ __forceinline__ void ns_gemm(int M, int N, int K, const float* A, int lda, const float* Bm, int ldb,
                                        float* C, int ldc, float alpha, float beta, const float* Cin, float diag,
                                        NsSmem& sm, int part = 0, int nparts = 1) {
  if (TC) {
    cta_gemm_mma<TRA, TRB>(M, N, K, A, lda, Bm, ldb, C, ldc, alpha, beta, Cin, diag, sm.t, part, nparts);
  } else {
    // the diagonal term is folded into the product by the CTA that owns the tile: added after its own tiles are stored
    cta_gemm<TRA, TRB>(M, N, K, A, lda, Bm, ldb, C, ldc, alpha, beta, Cin, sm.f, part, nparts);
    if (diag != 0.f) {
      const int lim = M < N ? M : N, tiles_n = (N + 63) / 64;
      for (int i = threadIdx.x; i < lim; i += 256)
        if (((i / 64) * tiles_n + i / 64) % nparts == part) C[(long long)i * ldc + i] += diag;
      __syncthreads();
    }
  }
}

// =====================================================================================
// Newton-Schulz forward for one m x m matrix (Alg. 2), whole CTA.
//   Wr <- W + eps I;  alpha = 1/(||Wr||_1 ||Wr||_inf) unless given;  X_0 = alpha Wr^T;
//   X_{k+1} = X_k (2I - Wr X_k);  Xh[k] = X_k for k = 0..T.
// W, Wr, P: [m][m] in global memory; Xh: [T+1][m][m].
// =====================================================================================
template <bool TC, int CL = 1>
__device__ void ns_forward_dev(int m, int T, float eps, float alpha_in, const float* W, float* Wr, float* P,
                               float* Xh, NsHdr* hdr, NsSmem& sm, float* red /* 2*256 + 8 floats */, int crank = 0,
                               float* Qh = nullptr) {
  // Qh: NULL, or a history [T][m][m] that keeps Q_k = 2I - Wr X_k for the adjoint (which then need not form Wr X_k again)
  // CL CTAs of a cluster share the work (crank = this CTA's rank): element-wise phases are strided over all their
  // threads, every product is split by output tiles, small reductions are done by each CTA for itself.
  const int tid = threadIdx.x, gt = crank * 256 + tid, gn = 256 * CL;
  const long long mm = (long long)m * m;
  for (long long e = gt; e < mm; e += gn) {
    const int i = (int)(e / m), j = (int)(e % m);
    Wr[e] = W[e] + (i == j ? eps : 0.f);
  }
  phase_sync<CL>();
  float* colsum = red;          // [256]
  float* rowsum = red + 256;    // [256]
  if (tid < m) {
    float cs = 0.f, rs = 0.f;
    for (int i = 0; i < m; ++i) { cs += fabsf(Wr[(long long)i * m + tid]); rs += fabsf(Wr[(long long)tid * m + i]); }
    colsum[tid] = cs; rowsum[tid] = rs;
  }
  __syncthreads();
  if (tid == 0) {               // every CTA of a cluster arrives at the same values
    float n1, ninf; int js, is;                   // near-ties (duplicated landmarks): the lowest index
    norm_argmax(colsum, m, n1, js);
    norm_argmax(rowsum, m, ninf, is);
    float* al = red + 512;
    al[0] = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * ninf);
    if (crank == 0) {
      hdr->n1 = n1; hdr->ninf = ninf; hdr->jstar = js; hdr->istar = is;
      hdr->auto_alpha = !(alpha_in > 0.f);
      hdr->alpha = al[0];
      hdr->pad0 = hdr->pad1 = 0;
    }
  }
  __syncthreads();
  const float alpha = red[512];
  for (long long e = gt; e < mm; e += gn) {
    const int i = (int)(e / m), j = (int)(e % m);
    Xh[e] = alpha * Wr[(long long)j * m + i];
  }
  phase_sync<CL>();
  for (int k = 0; k < T; ++k) {
    const float* X = Xh + (long long)k * mm;
    float* Xn = Xh + (long long)(k + 1) * mm;
    float* Q = Qh ? Qh + (long long)k * mm : P;
    ns_gemm<TC, false, false, true>(m, m, m, Wr, m, X, m, Q, m, -1.f, 0.f, nullptr, 2.f, sm, crank, CL);   // Q = 2I - Wr X_k
    if (CL > 1) phase_sync<CL>();
    ns_gemm<TC, false, false, true>(m, m, m, X, m, Q, m, Xn, m, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);    // X_{k+1} = X_k Q
    if (CL > 1) phase_sync<CL>();
  }
}

template <int CL, bool SYM = false>
__device__ void ns_backward_tail_dev(int m, const float* Wr, const NsHdr* hdr, const float* G, float* dW, float* red, int crank);

// =====================================================================================
// Exact adjoint of ns_forward_dev: given G0 = dLoss/dX_T returns dW = dLoss/dW.
// Scratch matrices [m][m]: P, Hm, Ga, Gb.  Xh holds X_0..X_T, Wr = W + eps I, hdr from the forward.
// =====================================================================================
template <bool TC, int CL = 1>
__device__ void ns_backward_dev(int m, int T, const float* Wr, const float* Xh, const NsHdr* hdr,
                                const float* G0, float* dW, float* P, float* Hm, float* Ga, float* Gb,
                                NsSmem& sm, float* red, int crank = 0, const float* Qh = nullptr) {
  // Qh: NULL, or the history of Q_k = 2I - Wr X_k the forward pass kept: 2G - G (Wr X_k)^T is then G Q_k^T, four
  // products per step instead of five
  const int tid = threadIdx.x, gt = crank * 256 + tid, gn = 256 * CL;
  const long long mm = (long long)m * m;
  for (long long e = gt; e < mm; e += gn) { Ga[e] = G0[e]; dW[e] = 0.f; }
  phase_sync<CL>();
  float* G = Ga; float* Gn = Gb;
  for (int k = T - 1; k >= 0; --k) {
    const float* A = Xh + (long long)k * mm;                                        // X_{k+1} = 2A - A P, P = Wr A
    if (!Qh) ns_gemm<TC, false, false, true>(m, m, m, Wr, m, A, m, P, m, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);      // P = Wr A
    ns_gemm<TC, true, false, true>(m, m, m, A, m, G, m, Hm, m, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);       // H = A^T G
    if (CL > 1) phase_sync<CL>();
    ns_gemm<TC, false, true, true>(m, m, m, Hm, m, A, m, dW, m, -1.f, 1.f, dW, 0.f, sm, crank, CL);          // dW -= H A^T
    if (Qh) ns_gemm<TC, false, true, true>(m, m, m, G, m, Qh + (long long)k * mm, m, Gn, m, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);   // Gn = G Q^T
    else ns_gemm<TC, false, true, true>(m, m, m, G, m, P, m, Gn, m, -1.f, 2.f, G, 0.f, sm, crank, CL);       // Gn = 2G - G P^T
    ns_gemm<TC, true, false, true>(m, m, m, Wr, m, Hm, m, Gn, m, -1.f, 1.f, Gn, 0.f, sm, crank, CL);         // Gn -= Wr^T H
    if (CL > 1) phase_sync<CL>();
    float* t = G; G = Gn; Gn = t;
  }
  ns_backward_tail_dev<CL>(m, Wr, hdr, G, dW, red, crank);
}

// End of the adjoint: X_0 = alpha Wr^T with alpha = 1 / (||Wr||_1 ||Wr||_inf) (unless given).  G = dLoss/dX_0 and dW
// (the part accumulated over the steps) are fp32 [m][m] in global memory; dW receives the rest.  CL CTAs share it.
// SYM: Wr is symmetric bit for bit (the landmark kernel matrix is), so <G, Wr^T> is read along the rows of both.
template <int CL, bool SYM>
__device__ void ns_backward_tail_dev(int m, const float* Wr, const NsHdr* hdr, const float* G, float* dW, float* red, int crank) {
  const int tid = threadIdx.x, gt = crank * 256 + tid, gn = 256 * CL;
  const long long mm = (long long)m * m;
  const float alpha = hdr->alpha;
  float part = 0.f;
  if (SYM) {
    float p4[4] = {0.f, 0.f, 0.f, 0.f};              // four independent chains: the loads of a batch overlap
    long long e = tid;
    for (; e + 3 * 256 < mm; e += 4 * 256) {
#pragma unroll
      for (int u = 0; u < 4; ++u) p4[u] += G[e + u * 256] * Wr[e + u * 256];
    }
    for (; e < mm; e += 256) p4[0] += G[e] * Wr[e];
    part = (p4[0] + p4[1]) + (p4[2] + p4[3]);
  } else {
    for (long long e = tid; e < mm; e += 256) {      // every CTA of a cluster sums everything (same order, same value)
      const int i = (int)(e / m), j = (int)(e % m);
      part += G[e] * Wr[(long long)j * m + i];
    }
  }
  const float dalpha = block_sum(part, red);
  for (long long e = gt; e < mm; e += gn) {
    const int j = (int)(e / m), i = (int)(e % m);      // dW[j][i] += alpha G[i][j]
    dW[e] += alpha * G[(long long)i * m + j];
  }
  phase_sync<CL>();
  if (hdr->auto_alpha) {
    const int js = hdr->jstar, is = hdr->istar;
    const float c1 = dalpha * (-alpha / hdr->n1), c2 = dalpha * (-alpha / hdr->ninf);
    if (crank == 0)
      for (int i = tid; i < m; i += 256) {
        const float w = Wr[(long long)i * m + js];
        dW[(long long)i * m + js] += c1 * (w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f));
      }
    __syncthreads();
    if (crank == 0)
      for (int j = tid; j < m; j += 256) {
        const float w = Wr[(long long)is * m + j];
        dW[(long long)is * m + j] += c2 * (w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f));
      }
    phase_sync<CL>();
  }
}

// End of the adjoint and the landmark-block factor in one pass, for a landmark matrix that is symmetric bit for bit
// (one landmark set) and was never written out with its ridge: Wr = W + eps I is formed where it is read.
//   dW_total = dWacc + alpha G^T + dalpha d(alpha)/dW,   dalpha = <G, Wr^T> = <G, Wr>,
//   GW = (dW_total o W + (dW_total o W)^T) / lambda = (F + F^T + E + E^T) o W / lambda,   F = dWacc + alpha G,
// E the two rank-one corrections of the norm gradient (column jstar of ||.||_1, row istar of ||.||_inf).  Transposed
// tiles go through shared memory (32 x 32, four per round); CL CTAs share the tiles.  G, dWacc: fp32 [m][m]; GW: [m][ldm],
// columns >= m zero.  tile: >= 4 * 32 * 33 + 512 floats of shared memory.
template <int CL>
__device__ void ns_tail_gw_sym(int m, int ldm, const float* __restrict__ W, float eps, const NsHdr* hdr, const float* __restrict__ G,
                               const float* __restrict__ dWacc, float inv_lambda, float* __restrict__ GW, float* red, float* tile, int crank) {
  const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  const unsigned mm = (unsigned)m * (unsigned)m, dstep = (unsigned)m + 1u;
  const float alpha = hdr->alpha;
  const int js = hdr->jstar, is = hdr->istar;
  float* sgc = tile + 4 * 32 * 33;          // sign of column jstar of Wr
  float* sgr = sgc + 256;                   // sign of row istar of Wr
  for (int i = tid; i < m; i += 256) {
    const float wc = W[(long long)i * m + js] + (i == js ? eps : 0.f), wr = W[(long long)is * m + i] + (i == is ? eps : 0.f);
    sgc[i] = wc > 0.f ? 1.f : (wc < 0.f ? -1.f : 0.f);
    sgr[i] = wr > 0.f ? 1.f : (wr < 0.f ? -1.f : 0.f);
  }
  float p16[16];
#pragma unroll
  for (int u = 0; u < 16; ++u) p16[u] = 0.f;
  unsigned e = (unsigned)tid;
  for (; e + 15u * 256u < mm; e += 16u * 256u) {      // every CTA sums everything (same order, same value)
    float g[16], w[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) { g[u] = G[e + u * 256u]; w[u] = W[e + u * 256u]; }
#pragma unroll
    for (int u = 0; u < 16; ++u) p16[u] += g[u] * (w[u] + ((e + u * 256u) % dstep == 0u ? eps : 0.f));
  }
  for (; e < mm; e += 256u) p16[0] += G[e] * (W[e] + (e % dstep == 0u ? eps : 0.f));
#pragma unroll
  for (int o = 8; o > 0; o >>= 1)
#pragma unroll
    for (int u = 0; u < o; ++u) p16[u] += p16[u + o];
  const float dalpha = block_sum(p16[0], red);          // ends with a barrier: sgc / sgr are complete as well
  const float c1 = hdr->auto_alpha ? dalpha * (-alpha / hdr->n1) : 0.f, c2 = hdr->auto_alpha ? dalpha * (-alpha / hdr->ninf) : 0.f;
  const int nti = (m + 31) / 32, ntj = (ldm + 31) / 32, ntiles = nti * ntj;
  constexpr int NT = 4;                      // tiles per round: their loads are in flight together
  for (int t0 = crank; t0 < ntiles; t0 += NT * CL) {
    float f[NT][4], w[NT][4], ft[NT][4];
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      const int t = t0 + q * CL, I = t / ntj, J = t % ntj;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = I * 32 + ty + 8 * r, j = J * 32 + tx;            // this thread's element of the tile
        const int jj = J * 32 + ty + 8 * r, ii = I * 32 + tx;          // and of the mirrored tile
        const bool in = t < ntiles && i < m && j < m, tin = t < ntiles && jj < m && ii < m;
        f[q][r] = in ? dWacc[(long long)i * m + j] : 0.f;
        ft[q][r] = in ? G[(long long)i * m + j] : 0.f;
        w[q][r] = in ? W[(long long)i * m + j] : 0.f;
        const float a = tin ? dWacc[(long long)jj * m + ii] : 0.f, b = tin ? G[(long long)jj * m + ii] : 0.f;
        f[q][r] = fmaf(alpha, ft[q][r], f[q][r]);
        ft[q][r] = fmaf(alpha, b, a);
      }
    }
    __syncthreads();                                                   // the tiles of the previous round have been read
#pragma unroll
    for (int q = 0; q < NT; ++q)
#pragma unroll
      for (int r = 0; r < 4; ++r) tile[q * (32 * 33) + (ty + 8 * r) * 33 + tx] = ft[q][r];
    __syncthreads();
#pragma unroll
    for (int q = 0; q < NT; ++q) {
      const int t = t0 + q * CL, I = t / ntj, J = t % ntj;
      if (t >= ntiles) continue;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = I * 32 + ty + 8 * r, j = J * 32 + tx;
        if (i >= m || j >= ldm) continue;
        float sum = f[q][r] + tile[q * (32 * 33) + tx * 33 + ty + 8 * r];
        if (j < m) {
          if (j == js) sum += c1 * sgc[i];
          if (i == is) sum += c2 * sgr[j];
          if (i == js) sum += c1 * sgc[j];
          if (j == is) sum += c2 * sgr[i];
        }
        GW[(long long)i * ldm + j] = (j < m) ? sum * w[q][r] * inv_lambda : 0.f;
      }
    }
  }
}

// =====================================================================================
// Conjugate gradients (the other solver of Sec. 5.3 / Table 4) for one head, whole CTA (256 threads):
//   X = the T-step iterate of (W + eps I) X = B from X_0 = 0, one independent solve per column of B [m][D]
//   (Hestenes-Stiefel: a = r.r / p.(Wr p), x += a p, r -= a Wr p, b = r'.r' / r.r, p = r' + b p).
// A column whose residual is exactly zero, or whose curvature p.(Wr p) is not positive, stops moving.
// The recurrence runs in DOUBLE precision: in single precision the iterates drift from the exact-arithmetic ones by
// 1e-4 after three steps and 3e-2 after four on the landmark matrices of this path (the directions lose their
// conjugacy), although the iterate itself depends on W and B only mildly; the inputs stay fp32.
// W: fp32 [m][m] without the ridge; Bsrc: fp32 [m][D]; Xout: fp32 [m][D]; scratch: 4 m D doubles (x, r, p, Wr p).
// Thread t always works on column t % D (256 % D == 0); the dot products of a column are added over the 256 / D
// threads that share it in a fixed order.  red: >= 2 * 256 + 8 floats; gsm: >= 18 KiB of shared memory.
// =====================================================================================
// Q = (W + eps I) P in double on the FP64 tensor-core instruction (mma.sync m8n8k4; plain DFMA runs at 8 per clock
// and SM on this part, a sixteenth of the FP32 rate, and bound the solver): 64 x 64 output tiles, K in chunks of 16
// staged in shared memory; warp w owns rows 32 (w / 4) .. + 31 and columns 16 (w % 4) .. + 15 of the tile, i.e. 4 x 2
// fragments of 8 x 8.  Fragment layout of the instruction: lane T holds A[T / 4][T % 4], B[T % 4][T / 4] and
// C[T / 4][2 (T % 4)], C[T / 4][2 (T % 4) + 1].
__device__ __forceinline__ void dmma884(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(c[0]), "+d"(c[1]) : "d"(a), "d"(b));
}
template <int D>
__device__ void cg_matvec(int m, float eps, const float* __restrict__ W, const double* __restrict__ P, double* __restrict__ Q, double* gsm) {
  constexpr int PA = 17, PB = 72;                                      // pitches (doubles): conflict-free fragment reads
  double* As = gsm;                                                    // [64][PA]: As[i][kk] = Wr[i0 + i][k0 + kk]
  double* Bs = gsm + 64 * PA;                                          // [16][PB]: Bs[kk][j] = P[k0 + kk][j0 + j]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, lr = lane >> 2, lc = lane & 3;
  const int wr = (warp >> 2) * 32, wc = (warp & 3) * 16;
  for (int i0 = 0; i0 < m; i0 += 64)
    for (int j0 = 0; j0 < D; j0 += 64) {
      double acc[4][2][2];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
      for (int k0 = 0; k0 < m; k0 += 16) {
        __syncthreads();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int e = tid + 256 * u;
          { const int i = e >> 4, kk = e & 15, gi = i0 + i, gk = k0 + kk;                 // consecutive threads along k
            As[i * PA + kk] = (gi < m && gk < m) ? (double)W[(long long)gi * m + gk] + (gi == gk ? (double)eps : 0.0) : 0.0; }
          { const int kk = e >> 6, j = e & 63, gk = k0 + kk, gj = j0 + j;
            Bs[kk * PB + j] = (gk < m && gj < D) ? P[(long long)gk * D + gj] : 0.0; }
        }
        __syncthreads();
#pragma unroll
        for (int k4 = 0; k4 < 16; k4 += 4) {
          double af[4], bf[2];
#pragma unroll
          for (int a = 0; a < 4; ++a) af[a] = As[(wr + 8 * a + lr) * PA + k4 + lc];
#pragma unroll
          for (int b = 0; b < 2; ++b) bf[b] = Bs[(k4 + lc) * PB + wc + 8 * b + lr];
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 2; ++b) dmma884(acc[a][b], af[a], bf[b]);
        }
      }
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int gi = i0 + wr + 8 * a + lr;
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          const int gj = j0 + wc + 8 * b + 2 * lc;
          if (gi < m && gj < D) Q[(long long)gi * D + gj] = acc[a][b][0];
          if (gi < m && gj + 1 < D) Q[(long long)gi * D + gj + 1] = acc[a][b][1];
        }
      }
    }
  __syncthreads();
}

template <int D>
__device__ void cg_dev(int m, int T, float eps, const float* W, const float* Bsrc, float* Xout, double* scratch, double* gsm, float* red) {
  constexpr int NG = 256 / D;
  const int tid = threadIdx.x, c = tid % D, md = m * D;
  // four disjoint arrays: the element-wise passes may keep several loads in flight
  double* __restrict__ X = scratch; double* __restrict__ R = scratch + md; double* __restrict__ P = scratch + 2 * md;
  double* __restrict__ Qv = scratch + 3 * md;
  double* dred = reinterpret_cast<double*>(red);     // [256] partial dot products (2 * 256 floats)
  __shared__ double rr_s[D], coef_s[D];
  __shared__ int frozen_s[D];
  auto column_sum = [&](double part) {               // sum over the threads of a column; valid in threads tid < D
    dred[tid] = part;
    __syncthreads();
    double t = 0.0;
    if (tid < D)
#pragma unroll
      for (int q = 0; q < NG; ++q) t += dred[q * D + tid];
    __syncthreads();
    return t;
  };
  double part = 0.0;
  for (int e = tid; e < md; e += 256) {
    const double b = (double)Bsrc[e];
    X[e] = 0.0; R[e] = b; P[e] = b;
    part += b * b;
  }
  {
    const double t = column_sum(part);
    if (tid < D) { rr_s[tid] = t; frozen_s[tid] = (t == 0.0) ? 1 : 0; }
  }
  __syncthreads();
  for (int k = 0; k < T; ++k) {
    cg_matvec<D>(m, eps, W, P, Qv, gsm);                                                 // Q = (W + eps I) P (ends with a barrier)
    part = 0.0;
#pragma unroll 4
    for (int e = tid; e < md; e += 256) part += P[e] * Qv[e];
    {
      const double pq = column_sum(part);
      if (tid < D) {
        if (!frozen_s[tid] && !(pq > 0.0)) frozen_s[tid] = 1;
        coef_s[tid] = frozen_s[tid] ? 0.0 : rr_s[tid] / pq;
      }
    }
    __syncthreads();
    const double a = coef_s[c];
    part = 0.0;
#pragma unroll 4
    for (int e = tid; e < md; e += 256) {
      X[e] = fma(a, P[e], X[e]);
      const double r = fma(-a, Qv[e], R[e]);
      R[e] = r;
      part += r * r;
    }
    {
      const double rn = column_sum(part);
      if (tid < D && !frozen_s[tid]) {
        coef_s[tid] = rn / rr_s[tid];
        rr_s[tid] = rn;
        if (rn == 0.0) frozen_s[tid] = 1;
      }
    }
    __syncthreads();
    if (!frozen_s[c]) {                              // a column that has stopped keeps its direction
      const double be = coef_s[c];
#pragma unroll 4
      for (int e = tid; e < md; e += 256) P[e] = fma(be, P[e], R[e]);
    }
    __syncthreads();
  }
  for (int e = tid; e < md; e += 256) Xout[e] = (float)X[e];
  __syncthreads();
}

// ------------------------------------------------------------------ stand-alone ns_pinv / ns_pinv_bwd
// CL CTAs of a thread-block cluster share a matrix (grid = batch * CL): every product is split by output tiles, the
// hardware cluster barrier ends a phase.  fp32 FFMA throughout (held to 2e-5 against the oracle).
template <int CL>
__global__ void __launch_bounds__(256) k_ns_pinv(int m, int T, float eps, float alpha_in, const float* W,
                                                 float* Wr, float* P, float* Xh, NsHdr* hdr, float* X,
                                                 float* resid) {
  __shared__ NsSmem sm;
  __shared__ float red[2 * 256 + 8];
  const int b = blockIdx.x / CL, crank = blockIdx.x % CL;
  const long long mm = (long long)m * m;
  W += b * mm; Wr += b * mm; P += b * mm; Xh += (long long)b * (T + 1) * mm; hdr += b;
  ns_forward_dev<false, CL>(m, T, eps, alpha_in, W, Wr, P, Xh, hdr, sm, red, crank);
  const float* XT = Xh + (long long)T * mm;
  if (X) for (long long e = crank * 256 + threadIdx.x; e < mm; e += 256 * CL) X[b * mm + e] = XT[e];
  if (resid) {
    ns_gemm<false, false, false>(m, m, m, Wr, m, XT, m, P, m, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);
    phase_sync<CL>();
    if (crank == 0) {
      float part = 0.f;
      for (long long e = threadIdx.x; e < mm; e += 256) {
        const int i = (int)(e / m), j = (int)(e % m);
        const float r = (i == j ? 1.f : 0.f) - P[e];
        part += r * r;
      }
      const float s = block_sum(part, red);
      if (threadIdx.x == 0) resid[b] = sqrtf(s);
    }
  }
  if (CL > 1) phase_sync<CL>();      // no CTA of the cluster leaves while another may still read what it wrote
}

// recompute != 0: run the forward first (Xh, hdr, Wr are scratch); else Xh is the caller's history
// and only Wr / hdr are rebuilt from W.
template <int CL>
__global__ void __launch_bounds__(256) k_ns_pinv_bwd(int m, int T, float eps, float alpha_in, const float* W,
                                                     float* Wr, float* P, float* Hm, float* Ga, float* Gb,
                                                     float* Xh_scratch, const float* Xh_given, NsHdr* hdr,
                                                     const float* dX, float* dW) {
  __shared__ NsSmem sm;
  __shared__ float red[2 * 256 + 8];
  const int b = blockIdx.x / CL, crank = blockIdx.x % CL;
  const long long mm = (long long)m * m;
  W += b * mm; Wr += b * mm; P += b * mm; Hm += b * mm; Ga += b * mm; Gb += b * mm; hdr += b;
  float* Xs = Xh_scratch + (long long)b * (T + 1) * mm;
  // T = 0 when the history is given: only Wr, the norms and alpha are rebuilt
  ns_forward_dev<false, CL>(m, Xh_given ? 0 : T, eps, alpha_in, W, Wr, P, Xs, hdr, sm, red, crank);
  const float* Xh = Xh_given ? Xh_given + (long long)b * (T + 1) * mm : Xs;
  ns_backward_dev<false, CL>(m, T, Wr, Xh, hdr, dX + b * mm, dW + b * mm, P, Hm, Ga, Gb, sm, red, crank);
  if (CL > 1) phase_sync<CL>();
}

// =====================================================================================
// Per-head middle of the forward pass: reduce M over the token chunks, Newton-Schulz, Y = X M,
// then fold the injective map (Prop. 3) into Ytilde_l = s_l Y_l - mean_l'(s_l' Y_l'), ybar = mean_l Y_l
// so that O = (C - mu) Ytilde + ybar.  One CTA per head.
// =====================================================================================
// MP: 0 = matrices in global memory (fp32 FFMA or the cluster-shared mma.sync engine); 64 / 128 = one CTA per head on
// tcgen05 with the matrix padded to MP; 256 = tcgen05 on 2 x 2 blocks of 128, CL = 2 CTAs of a thread-block cluster
// per head (grid = heads * CL).
template <int D, bool TC, int MP, int CL = 1>
__global__ void __launch_bounds__(256, MP == 64 ? 3 : ((CL > 1 && MP == 0) ? 2 : 1)) k_mid_fwd(int m, int ldm, int T, float eps, float alpha_in, int H, int map_mode,
                                                 const float* __restrict__ whiten, const float* W, float* Wr,
                                                 float* P, float* Xh, float* Ph, NsHdr* hdr, const float* Mpart, int nchunks,
                                                 float* Mout, float* Y, float* Yt, float* ybar, int* dev_status,
                                                 long long hslot, bf16* Yimg, int phase, int solver = 0, float* cgws = nullptr) {
  // solver: 0 = Newton-Schulz (Alg. 2) and Y = X_T M; 1 = conjugate gradients on (W + eps I) Y = M (Sec. 5.3, Table 4;
  // the single-CTA instantiation without tensor cores only), cgws = 4 m D doubles of scratch per head
  // phase: bit 0 = Newton-Schulz (needs W only), bit 1 = everything that needs M (sum of the partials, Y, map fold).
  // The two halves may run as two launches, the first beside the kernels that produce M; X_T passes through
  // global memory either way.
  // Yimg: NULL, or where Ytilde is also left as split operand images per 64-landmark block (for the tcgen05 product)
  // hslot: floats per slot of the iterate histories (the tcgen05 paths, whose slots hold operand images)
  // dynamic shared memory: the Newton-Schulz matrices (MP > 0), reused afterwards by the GEMM engine
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  NsSmem& sm = *reinterpret_cast<NsSmem*>(dyn_smem);
  __shared__ float red[2 * 256 + 8];
  const int bh = blockIdx.x / CL, crank = blockIdx.x % CL, tid = threadIdx.x;
  const int gt = crank * 256 + tid, gn = 256 * CL;      // this thread among all threads that share the head
  const long long mm = (long long)m * m, md = (long long)m * D;
  // X_T of the single-CTA tcgen05 paths uses the padded leading dimension (128-bit accesses)
  const int ldx = (MP == 64 || MP == 128) ? ldm : m;
  const long long mx = (MP > 0) ? hslot : (long long)m * ldx;
  const long long wslot = (MP == 256) ? kU2Slot : mm;           // floats per scratch matrix
  W += bh * mm; Wr += bh * wslot; P += bh * wslot; Xh += (long long)bh * (T + 1) * mx; hdr += bh;
  if (Ph) Ph += (long long)bh * T * mx;
  Mout += bh * md; Y += bh * md; Yt += bh * md; ybar += (long long)bh * D;
  Mpart += (long long)bh * nchunks * md;
  if ((phase & 2) && nchunks > 0)                // nchunks == 0: the single partial result was written to Mout directly
    // eight elements of this thread at a time: their loads of a part are in flight together, the parts in order
    for (long long e0 = (long long)gt * 4; e0 < md; e0 += 32ll * gn) {
      float4 acc[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int p = 0; p < nchunks; ++p) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const long long e = e0 + 4ll * u * gn;
          v[u] = e < md ? *reinterpret_cast<const float4*>(Mpart + (long long)p * md + e) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) { acc[u].x += v[u].x; acc[u].y += v[u].y; acc[u].z += v[u].z; acc[u].w += v[u].w; }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const long long e = e0 + 4ll * u * gn;
        if (e < md) *reinterpret_cast<float4*>(Mout + e) = acc[u];
      }
    }
  const float* XT = Xh + (long long)T * mx;
  // the 256-wide engine keeps one tensor-memory allocation for the iteration and the product Y = X_T M
  __shared__ UmmaCtl ctl256;
  __shared__ __align__(8) unsigned long long mbars256[3];
  U2Ctx u2c;
  if ((phase & 1) && solver == 0) {
  bool tc_ok = true;
  float bad = 0.f;                               // non-finite entries of X_T seen by this thread
  if constexpr (MP == 128 || MP == 64) {        // tcgen05 + TMEM, the matrix padded to MP x MP
    __shared__ UmmaCtl ctl;
    tc_ok = ns_forward_umma<MP>(m, T, eps, alpha_in, W, Xh, Ph, ldx, mx, hdr, reinterpret_cast<bf16*>(dyn_smem), red, ctl, bad);
    __syncthreads();
  } else if constexpr (MP == 256) {             // tcgen05 + TMEM, 2 x 2 blocks of 128 shared by the two CTAs of a cluster
    static_assert(MP != 256 || CL == kU2Cluster, "the 256-wide engine is written for its own cluster size");
    u2_begin(u2c, ctl256, mbars256, reinterpret_cast<bf16*>(dyn_smem), 256);
    tc_ok = ns_forward_umma256(u2c, m, T, eps, alpha_in, W, P, Wr, Xh, Ph, hdr, red, crank, bad);
    if (!(phase & 2)) umma_end(ctl256, 256);
    __syncthreads();
  } else {
    ns_forward_dev<TC, CL>(m, T, eps, alpha_in, W, Wr, P, Xh, hdr, sm, red, crank, Ph);
  }
  if (dev_status) {
    if constexpr (MP == 0)
      for (int e = tid; e < m * m; e += 256) bad += isfinite(XT[(long long)(e / m) * ldx + e % m]) ? 0.f : 1.f;
    bad = block_sum(bad, red);
    if (tid == 0 && crank == 0) atomicOr(dev_status + bh, (bad > 0.f ? 1 : 0) | (tc_ok ? 0 : 2));   // bit1: a bounded tensor-core wait ran out
  }
  }
  if (!(phase & 2)) return;
  if (!(phase & 1)) phase_sync<CL>();             // the M sums of all threads that share the head
  if (solver == 1) {
    if constexpr (!TC && MP == 0 && CL == 1) {
      __syncthreads();
      cg_dev<D>(m, T, eps, W, Mout, Y, reinterpret_cast<double*>(cgws) + (long long)bh * 4 * md, reinterpret_cast<double*>(dyn_smem), red);
      if (dev_status) {
        float bad = 0.f;
        for (int e = tid; e < m * D; e += 256) bad += isfinite(Y[e]) ? 0.f : 1.f;
        bad = block_sum(bad, red);
        if (tid == 0 && bad > 0.f) atomicOr(dev_status + bh, 1);
      }
    }
  } else if constexpr (MP == 256) {               // Y = X M on the engine of the iteration (images of X_T in Wr, of M in P)
    if (!(phase & 1)) u2_begin(u2c, ctl256, mbars256, reinterpret_cast<bf16*>(dyn_smem), 256);
    const bool y_ok = u2_product_y(u2c, m, D, Wr, Mout, P, Y, crank);
    umma_end(ctl256, 256);
    if (dev_status && !y_ok && tid == 0 && crank == 0) atomicOr(dev_status + bh, 2);
    phase_sync<CL>();
  } else {
    ns_gemm<TC, false, false>(m, D, m, XT, ldx, Mout, D, Y, D, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);   // Y = X M
    if (CL > 1) phase_sync<CL>();
  }
  const float* s = whiten ? whiten + (long long)(bh % H) * m : nullptr;
  // fold the injective map (Prop. 3): column means over the landmarks first (256 / D thread groups share the
  // landmarks of a column, eight independent loads per batch, the groups added in order), then every element in parallel
  float* colstat = red;            // [2][D]: mean_l s_l Y_lc and mean_l Y_lc
  {
    constexpr int NG = 256 / D;
    const int c = tid % D, g = tid / D;
    float sy = 0.f, y1 = 0.f;
    for (int l0 = g; l0 < m; l0 += 8 * NG) {
      float y[8], w[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int l = l0 + u * NG;
        y[u] = (l < m) ? Y[(long long)l * D + c] : 0.f;
        w[u] = (l < m && s) ? s[l] : 1.f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) { sy += w[u] * y[u]; y1 += y[u]; }
    }
    red[tid] = sy; red[256 + tid] = y1;
    __syncthreads();
    if (tid < D) {                 // thread tid reads, then overwrites, slots that only it touches
      sy = 0.f; y1 = 0.f;
#pragma unroll
      for (int q = 0; q < NG; ++q) { sy += red[q * D + tid]; y1 += red[256 + q * D + tid]; }
      colstat[tid] = sy / (float)m;
      colstat[D + tid] = y1 / (float)m;
      if (crank == 0) ybar[tid] = (map_mode == 1) ? y1 / (float)m : 0.f;
    }
  }
  __syncthreads();
  for (long long e = (long long)gt * 4; e < md; e += 4 * gn) {
    const int l = (int)(e / D), c = (int)(e % D);
    float4 y = *reinterpret_cast<const float4*>(Y + e);
    if (map_mode == 1) {
      const float sl = s ? s[l] : 1.f;
      y.x = sl * y.x - colstat[c]; y.y = sl * y.y - colstat[c + 1];
      y.z = sl * y.z - colstat[c + 2]; y.w = sl * y.w - colstat[c + 3];
    }
    *reinterpret_cast<float4*>(Yt + e) = y;
  }
  if (Yimg != nullptr) {
    phase_sync<CL>();                             // Ytilde of this head is complete
    const int nkb = (m + GU_KB - 1) / GU_KB;
    gu_write_images(Yt, Yimg + (long long)bh * nkb * (2 * GU_KB * D), m, D, gt, gn);
  }
}
template <int D, bool TC, int MP, int CL = 1>
__global__ void __launch_bounds__(256, MP == 64 ? 3 : ((CL > 1 && MP == 0) ? 2 : 1)) k_mid_bwd(int m, int T, int H, int map_mode, float inv_lambda, int ldm,
                                                 const float* __restrict__ whiten, const float* W,
                                                 const float* Xh, const float* Ph, const NsHdr* hdr, const float* Msaved,
                                                 const float* dYtpart, const float* dybpart, int nchunks,
                                                 float eps, float* Wr, float* P, float* Hm, float* Ga, float* Gb,
                                                 float* dWm, float* dXm, float* dY, float* dM, float* GW, int* dev_status,
                                                 long long hslot, bf16* dMimg, int sym, int solver = 0, const float* Ysaved = nullptr,
                                                 float* cgws = nullptr, int phase = 3) {
  // phase: bit 0 = dY, dX and dM (what the key-side kernels wait for), bit 1 = the adjoint of the iteration and GW.
  // The two halves may run as two launches on one stream: the key-side sign pass then starts after the first.
  // solver 1 (conjugate gradients, the fp32 single-CTA instantiation only): the solve is differentiated as the linear
  // system it approximates, dM = the T-step iterate of (W + eps I) dM = dY, dW = -dM Y^T (Ysaved: Y of the forward pass)
  // sym: 1 = one landmark set (W = k(L, L): the gradient of both roles of L is carried by the symmetrised factor);
  // 0 = two landmark sets, GW = dW o W / lambda as it is (MP == 0 only)
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  NsSmem& sm = *reinterpret_cast<NsSmem*>(dyn_smem);
  __shared__ float red[2 * 256 + 8];
  const int bh = blockIdx.x / CL, crank = blockIdx.x % CL, tid = threadIdx.x;
  const int gt = crank * 256 + tid, gn = 256 * CL;
  const long long mm = (long long)m * m, md = (long long)m * D;
  const int ldx = (MP == 64 || MP == 128) ? ldm : m;
  const long long mx = (MP > 0) ? hslot : (long long)m * ldx;          // one slot of the iterate histories
  const long long ms = (MP == 256) ? kU2Slot : (long long)m * ldm;     // one scratch matrix
  W += bh * mm; Xh += (long long)bh * (T + 1) * mx; Ph += (long long)bh * T * mx; hdr += bh; Msaved += bh * md;
  Wr += bh * ms; P += bh * ms; Hm += bh * ms; Ga += bh * ms; Gb += bh * ms; dWm += bh * ms; dXm += bh * ms;
  dY += bh * md; dM += bh * md; GW += (long long)bh * m * ldm;
  dYtpart += (long long)bh * nchunks * md; dybpart += (long long)bh * nchunks * D;
  const float* s = whiten ? whiten + (long long)(bh % H) * m : nullptr;
  // the 256-wide engine keeps one tensor-memory allocation for the products in front of the adjoint and the adjoint
  __shared__ UmmaCtl ctl256;
  __shared__ __align__(8) unsigned long long mbars256[3];
  U2Ctx u2c;
  if (phase & 1) {
  float* dyb = red;   // [D] column sums of dO
  if (tid < D) {
    float t = 0.f;
    for (int p = 0; p < nchunks; ++p) t += dybpart[(long long)p * D + tid];
    dyb[tid] = t;
  }
  __syncthreads();
  // eight elements of this thread at a time: their loads of a part are in flight together, the parts in order
  for (long long e0 = (long long)gt * 4; e0 < md; e0 += 32ll * gn) {
    float4 acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int p = 0; p < nchunks; ++p) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const long long e = e0 + 4ll * u * gn;
        v[u] = e < md ? *reinterpret_cast<const float4*>(dYtpart + (long long)p * md + e) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) { acc[u].x += v[u].x; acc[u].y += v[u].y; acc[u].z += v[u].z; acc[u].w += v[u].w; }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const long long e = e0 + 4ll * u * gn;
      if (e >= md) continue;
      const float4 t = acc[u];
      const int l = (int)(e / D), c = (int)(e % D);
      // Ytilde = P_c diag(s) Y, ybar = Y^T 1/m  ->  dY = diag(s) (centred Z'^T dO) + (1/m) 1 dyb^T
      float4 o = t;
      if (map_mode == 1) {
        const float sl = s ? s[l] : 1.f, im = 1.f / (float)m;
        o.x = sl * t.x + dyb[c] * im; o.y = sl * t.y + dyb[c + 1] * im;
        o.z = sl * t.z + dyb[c + 2] * im; o.w = sl * t.w + dyb[c + 3] * im;
      }
      *reinterpret_cast<float4*>(dY + e) = o;
    }
  }
  if constexpr (MP == 0) {                          // m <= 256: 32-bit index arithmetic (a 64-bit division costs far more)
    for (unsigned e = (unsigned)gt; e < (unsigned)mm; e += (unsigned)gn) Wr[e] = W[e] + (e % (unsigned)(m + 1) == 0u ? eps : 0.f);
  }
  phase_sync<CL>();
  const float* XT = Xh + (long long)T * mx;
  if (solver == 1) {
    if constexpr (!TC && MP == 0 && CL == 1) {
      cg_dev<D>(m, T, eps, W, dY, dM, reinterpret_cast<double*>(cgws) + (long long)bh * 4 * md, reinterpret_cast<double*>(dyn_smem), red);
      ns_gemm<TC, false, true>(m, m, D, dM, D, Ysaved + bh * md, D, dWm, ldx, -1.f, 0.f, nullptr, 0.f, sm, crank, CL);   // dW = -dM Y^T
    }
  } else if constexpr (MP == 256) {                  // dX = dY M^T and dM = X^T dY on the engine of the adjoint
    u2_begin(u2c, ctl256, mbars256, reinterpret_cast<bf16*>(dyn_smem), 512);
    const bool p_ok = u2_products_dx_dm(u2c, m, D, dY, Msaved, XT, Hm, Gb, dXm, dM, crank);
    if (!(phase & 2)) umma_end(ctl256, 512);
    if (dev_status && !p_ok && tid == 0 && crank == 0) atomicOr(dev_status + bh, 2);
  } else {
    ns_gemm<TC, false, true>(m, m, D, dY, D, Msaved, D, dXm, ldx, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);   // dX = dY M^T
    ns_gemm<TC, true, false>(m, D, m, XT, ldx, dY, D, dM, D, 1.f, 0.f, nullptr, 0.f, sm, crank, CL);        // dM = X^T dY
  }
  if (CL > 1 && MP != 256) phase_sync<CL>();
  if (dMimg != nullptr) {                         // dM also as split operand images (for the tcgen05 product dV = R^T dM)
    const int nkb = (m + GU_KB - 1) / GU_KB;
    gu_write_images(dM, dMimg + (long long)bh * nkb * (2 * GU_KB * D), m, D, gt, gn);
  }
  }
  if (!(phase & 2)) return;
  if constexpr (MP == 128 || MP == 64) {
    __shared__ UmmaCtl ctl;
    const bool tc_ok = ns_backward_umma<MP>(m, T, eps, W, Xh, Ph, ldx, mx, hdr, dXm, GW, ldm, inv_lambda, reinterpret_cast<bf16*>(dyn_smem), red, ctl);
    if (dev_status && !tc_ok && tid == 0) atomicOr(dev_status + bh, 2);
  } else if constexpr (MP == 256) {
    if (!(phase & 1)) u2_begin(u2c, ctl256, mbars256, reinterpret_cast<bf16*>(dyn_smem), 512);
    const bool tc_ok = ns_backward_umma256(u2c, m, T, Xh, Ph, dXm, Ga, Gb, Hm, Wr, P, dWm, crank);
    umma_end(ctl256, 512);
    if (dev_status && !tc_ok && tid == 0 && crank == 0) atomicOr(dev_status + bh, 2);
    // end of the adjoint and GW in one pass (the operand buffers are free: the engine has ended with a cluster barrier)
    ns_tail_gw_sym<CL>(m, ldm, W, eps, hdr, P, dWm, inv_lambda, GW, red, reinterpret_cast<float*>(dyn_smem), crank);
  } else if (solver == 0) { ns_backward_dev<TC, CL>(m, T, Wr, Xh, hdr, dXm, dWm, P, Hm, Ga, Gb, sm, red, crank, Ph); if (CL > 1) phase_sync<CL>(); }
  // GW = (dW o K_LL + (dW o K_LL)^T) / lambda; four elements per batch so that the loads overlap
  // (the tcgen05 engines have written GW already)
  if constexpr (MP == 0)
  for (long long e0 = (long long)gt * 4; e0 < (long long)m * ldm; e0 += 4 * gn) {
    float a[4], b[4], c[4], d4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long e = e0 + u;
      const int i = (int)(e / ldm), j = (int)(e % ldm);
      const bool in = j < m;
      a[u] = in ? dWm[(long long)i * ldx + j] : 0.f;  b[u] = in ? W[(long long)i * m + j] : 0.f;
      c[u] = (in && sym) ? dWm[(long long)j * ldx + i] : 0.f;  d4[u] = (in && sym) ? W[(long long)j * m + i] : 0.f;
    }
    *reinterpret_cast<float4*>(GW + e0) = make_float4((a[0] * b[0] + c[0] * d4[0]) * inv_lambda, (a[1] * b[1] + c[1] * d4[1]) * inv_lambda,
                                                      (a[2] * b[2] + c[2] * d4[2]) * inv_lambda, (a[3] * b[3] + c[3] * d4[3]) * inv_lambda);
  }
}

// =====================================================================================
// Self-test of the bounded wait every tensor-core kernel of this library uses: an mbarrier on which nothing ever
// arrives is waited for with a probe limit; the wait must give up, and the kernel reports it the way the product
// kernels do (bit 1 of the status word) and returns normally.
// =====================================================================================
__global__ void k_selftest_wait(int probes, int* dev_status) {
  __shared__ __align__(8) unsigned long long mbar;
  if (threadIdx.x == 0) umma::mbar_init(&mbar, 1);
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = umma::mbar_wait(&mbar, 0, probes);
    if (!ok) atomicOr(dev_status, 2);
  }
}

// =====================================================================================
// FP32 add-rate probe: every thread runs kProbeChains independent chains of dependent adds, two lanes per chain and
// step (mode 0: two scalar adds, mode 1: one packed add.f32x2), no memory traffic inside the loop.  The rate it
// sustains is the measured counterpart of the derived lane-operation peak (SMs x 128 lanes x clock) that the
// l1 kernels are held against.
// =====================================================================================
constexpr int kProbeChains = 8;
// mode 0: two scalar adds per chain and step; 1: one packed add; 2: the instruction mix of the sign pass (two saturating
// multiply-adds that form a pair h, then two packed multiply-adds g h + acc into two accumulators: 6 lane-operations
// in 4 instructions); 3: the mix of the l1 forward (one packed subtract, two scalar |.| accumulations: 4 lane-operations
// in 3 instructions); 4: mix 2 with scalar and packed instructions in separate runs; 5: mix 2 with scalar instructions
// only.  Lane-operations per chain and step: 2, 2, 6, 4, 6, 6.
__global__ void __launch_bounds__(256) k_fp32_add_probe(int iters, int mode, float* sink) {
  const float x = sink[0];                       // a run-time value the compiler cannot fold
  float a[kProbeChains], b[kProbeChains];
#pragma unroll
  for (int k = 0; k < kProbeChains; ++k) { a[k] = (float)k; b[k] = (float)(k + threadIdx.x); }
  if (mode == 0) {
#pragma unroll 4
    for (int i = 0; i < iters; ++i)
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) { a[k] += x; b[k] += x; }
  } else if (mode == 1) {
    f32x2 v[kProbeChains];
    const f32x2 xx = pack2(x, x);
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) v[k] = pack2(a[k], b[k]);
#pragma unroll 4
    for (int i = 0; i < iters; ++i)
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) v[k] = add2(v[k], xx);
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { a[k] = lo32(v[k]); b[k] = hi32(v[k]); }
  } else if (mode == 2) {
    f32x2 r[kProbeChains], c[kProbeChains];
    const f32x2 gg = pack2(x, x + 1.f);
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { r[k] = pack2(a[k], b[k]); c[k] = pack2(b[k], a[k]); }
#pragma unroll 4
    for (int i = 0; i < iters; ++i)
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) {
        const f32x2 h = sat_fma_pair(lo32(r[k]), hi32(c[k]), x, 0.25f);     // inputs change every step: nothing can be hoisted
        r[k] = fma2(gg, h, r[k]);
        c[k] = fma2(gg, h, c[k]);
      }
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { a[k] = lo32(r[k]) + hi32(c[k]); b[k] = hi32(r[k]) + lo32(c[k]); }
  } else if (mode == 4) {      // the sign-pass mix with the scalar and the packed instructions in separate runs of 16
    f32x2 r[kProbeChains], c[kProbeChains];
    const f32x2 gg = pack2(x, x + 1.f);
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { r[k] = pack2(a[k], b[k]); c[k] = pack2(b[k], a[k]); }
#pragma unroll 2
    for (int i = 0; i < iters; ++i) {
      f32x2 h[kProbeChains];
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) h[k] = sat_fma_pair(lo32(r[k]), hi32(c[k]), x, 0.25f);
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) r[k] = fma2(gg, h[k], r[k]);
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) c[k] = fma2(gg, h[k], c[k]);
    }
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { a[k] = lo32(r[k]) + hi32(c[k]); b[k] = hi32(r[k]) + lo32(c[k]); }
  } else if (mode == 5) {      // the same arithmetic with scalar instructions only (two saturating and four plain multiply-adds)
    float r0[kProbeChains], r1[kProbeChains], c0[kProbeChains], c1[kProbeChains];
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { r0[k] = a[k]; r1[k] = b[k]; c0[k] = b[k]; c1[k] = a[k]; }
    const float g0 = x, g1 = x + 1.f;
#pragma unroll 4
    for (int i = 0; i < iters; ++i)
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) {
        const float h0 = sat_fma(r0[k], x, 0.25f), h1 = sat_fma(c1[k], x, 0.25f);
        r0[k] = fmaf(g0, h0, r0[k]); r1[k] = fmaf(g1, h1, r1[k]);
        c0[k] = fmaf(g0, h0, c0[k]); c1[k] = fmaf(g1, h1, c1[k]);
      }
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { a[k] = r0[k] + c1[k]; b[k] = r1[k] + c0[k]; }
  } else {
    const f32x2 nb = pack2(-x, -x - 1.f);
    f32x2 q[kProbeChains];
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) q[k] = pack2(a[k], b[k]);
    float acc[kProbeChains];
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) acc[k] = 0.f;
#pragma unroll 4
    for (int i = 0; i < iters; ++i)
#pragma unroll
      for (int k = 0; k < kProbeChains; ++k) {
        const f32x2 t = add2(q[k], nb);
        q[k] = t;                                                            // the operand changes every step
        acc[k] += fabsf(lo32(t));
        acc[k] += fabsf(hi32(t));
      }
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) { a[k] = acc[k]; b[k] = lo32(q[k]); }
  }
  float t = 0.f;
#pragma unroll
  for (int k = 0; k < kProbeChains; ++k) t += a[k] + b[k];
  if (t == 123456.789f) sink[1 + (blockIdx.x * 256 + threadIdx.x) % 1024] = t;    // practically never: keeps the chains alive
}

}  // namespace ln
