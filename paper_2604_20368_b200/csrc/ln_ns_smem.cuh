// Newton-Schulz (Alg. 2) and its adjoint with every m x m matrix resident in shared memory as
// bf16 hi + lo, multiplied on tensor cores (mma.sync, three MMAs per product, fp32 accumulators
// in registers).  One CTA of 256 threads per head.  Only the fp32 iterates X_k that the backward
// pass needs go to global memory.  MP is m padded to 64 or 128; padding rows and columns are zero
// and stay zero through the iteration (X_0 = alpha W^T has zero padding, and a zero row or column
// of X gives a zero row or column of X (2I - W X)).
#pragma once
#include "ln_mma.cuh"

namespace ln {

template <int MP> struct NsTile {
  static constexpr int LD = MP + 8;                 // bf16 elements per row (16-byte multiple, conflict-free ldmatrix)
  static constexpr int MT = MP / 64;                // m16 tiles per warp
  static constexpr int NT = MP / 16;                // n8 tiles per warp
  static constexpr int MAT = MP * LD;               // bf16 elements of one matrix part (hi or lo)
  static constexpr size_t mat_bytes = (size_t)2 * MAT * sizeof(bf16);   // hi + lo
  __device__ static __forceinline__ int wm() { return ((threadIdx.x >> 5) & 3) * (MP / 4); }
  __device__ static __forceinline__ int wn() { return (threadIdx.x >> 7) * (MP / 2); }
};

// acc (+)= op(A) op(B), all MP x MP, operands in shared memory (hi at p, lo at p + MAT).
//   TRA = false: A stored [M][K];  true: stored [K][M] (A^T is used)
//   TRB = false: B stored [K][N];  true: stored [N][K] (B^T is used)
template <int MP, bool TRA, bool TRB>
__device__ __forceinline__ void smem_gemm(float (&acc)[NsTile<MP>::MT][NsTile<MP>::NT][4], const bf16* A, const bf16* Bm,
                                          bool accumulate) {
  using TL = NsTile<MP>;
  constexpr int LD = TL::LD, MT = TL::MT, NT = TL::NT, MAT = TL::MAT;
  const int wm = TL::wm(), wn = TL::wn();
  if (!accumulate) {
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[a][t][q] = 0.f;
  }
  // all fragments of a k-step are fetched before its MMAs are issued, so the loads of the next
  // step overlap the tensor-core work of this one
#pragma unroll 2
  for (int k0 = 0; k0 < MP; k0 += 16) {
    uint32_t ah[MT][4], al[MT][4], bh4[NT / 2][4], bl4[NT / 2][4];
#pragma unroll
    for (int a = 0; a < MT; ++a) {
      if (TRA) { ldsm_x4_t(ah[a], addr_at(A, LD, k0, wm + a * 16)); ldsm_x4_t(al[a], addr_at(A + MAT, LD, k0, wm + a * 16)); }
      else     { ldsm_x4(ah[a], addr_a(A, LD, wm + a * 16, k0));    ldsm_x4(al[a], addr_a(A + MAT, LD, wm + a * 16, k0)); }
    }
#pragma unroll
    for (int t = 0; t < NT / 2; ++t) {
      if (TRB) { ldsm_x4(bh4[t], addr_b(Bm, LD, wn + t * 16, k0));    ldsm_x4(bl4[t], addr_b(Bm + MAT, LD, wn + t * 16, k0)); }
      else     { ldsm_x4_t(bh4[t], addr_bt(Bm, LD, k0, wn + t * 16)); ldsm_x4_t(bl4[t], addr_bt(Bm + MAT, LD, k0, wn + t * 16)); }
    }
    // three passes (lo*hi, hi*lo, hi*hi) so that consecutive MMAs hit different accumulators
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int t = 0; t < NT / 2; ++t) {
        mma_bf16(acc[a][2 * t], al[a], bh4[t][0], bh4[t][1]);
        mma_bf16(acc[a][2 * t + 1], al[a], bh4[t][2], bh4[t][3]);
      }
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int t = 0; t < NT / 2; ++t) {
        mma_bf16(acc[a][2 * t], ah[a], bl4[t][0], bl4[t][1]);
        mma_bf16(acc[a][2 * t + 1], ah[a], bl4[t][2], bl4[t][3]);
      }
#pragma unroll
    for (int a = 0; a < MT; ++a)
#pragma unroll
      for (int t = 0; t < NT / 2; ++t) {
        mma_bf16(acc[a][2 * t], ah[a], bh4[t][0], bh4[t][1]);
        mma_bf16(acc[a][2 * t + 1], ah[a], bh4[t][2], bh4[t][3]);
      }
  }
}

// Coordinates of accumulator element q of tile (a, t) of this thread.
template <int MP> __device__ __forceinline__ void frag_ij(int a, int t, int q, int& i, int& j) {
  const int lane = threadIdx.x & 31;
  i = NsTile<MP>::wm() + a * 16 + (lane >> 2) + (q >> 1) * 8;
  j = NsTile<MP>::wn() + t * 8 + 2 * (lane & 3) + (q & 1);
}

// registers (fragment layout) -> shared hi/lo matrix
template <int MP>
__device__ __forceinline__ void frag_to_smem(const float (&acc)[NsTile<MP>::MT][NsTile<MP>::NT][4], bf16* dst) {
  using TL = NsTile<MP>;
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        int i, j;
        frag_ij<MP>(a, t, 2 * h, i, j);
        bf16 h0, l0, h1, l1;
        split2(acc[a][t][2 * h], h0, l0);
        split2(acc[a][t][2 * h + 1], h1, l1);
        *reinterpret_cast<uint32_t*>(dst + i * TL::LD + j) =
            (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        *reinterpret_cast<uint32_t*>(dst + TL::MAT + i * TL::LD + j) =
            (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
      }
}

// registers (fragment layout) -> global fp32 [m][m]
template <int MP>
__device__ __forceinline__ void frag_to_global(const float (&acc)[NsTile<MP>::MT][NsTile<MP>::NT][4], float* dst, int m) {
  using TL = NsTile<MP>;
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int i, j;
        frag_ij<MP>(a, t, q, i, j);
        if (i < m && j < m) dst[(long long)i * m + j] = acc[a][t][q];
      }
}

// global fp32 [m][m] (+ diag on the diagonal, times scale, optionally transposed) -> shared hi/lo, zero padded.
// Eight independent loads are issued before anything is stored, so their latencies overlap.
template <int MP>
__device__ __forceinline__ void global_to_smem(const float* __restrict__ src, int m, float diag, float scale, bool transpose,
                                               bf16* dst) {
  using TL = NsTile<MP>;
  constexpr int PER = MP * MP / 256;       // elements per thread
#pragma unroll 1
  for (int b0 = 0; b0 < PER; b0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = (b0 + u) * 256 + threadIdx.x, i = e / MP, j = e % MP;
      float x = 0.f;
      if (i < m && j < m) {
        x = transpose ? src[(long long)j * m + i] : src[(long long)i * m + j];
        if (i == j) x += diag;
        x *= scale;
      }
      v[u] = x;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = (b0 + u) * 256 + threadIdx.x, i = e / MP, j = e % MP;
      bf16 h, l;
      split2(v[u], h, l);
      dst[i * TL::LD + j] = h;
      dst[TL::MAT + i * TL::LD + j] = l;
    }
  }
}

// Row / column absolute sums of W + eps I, alpha and the arg-max indices (lowest index on ties).
__device__ inline void ns_norms(int m, float eps, float alpha_in, const float* W, NsHdr* hdr, float* red /* >= 512 floats */) {
  const int tid = threadIdx.x;
  float* colsum = red;
  float* rowsum = red + 256;
  if (tid < m) {
    float cs = 0.f, rs = 0.f;
    for (int i = 0; i < m; ++i) {
      cs += fabsf(W[(long long)i * m + tid] + (i == tid ? eps : 0.f));
      rs += fabsf(W[(long long)tid * m + i] + (i == tid ? eps : 0.f));
    }
    colsum[tid] = cs; rowsum[tid] = rs;
  }
  __syncthreads();
  if (tid == 0) {
    float n1 = -1.f, ninf = -1.f; int js = 0, is = 0;
    for (int t = 0; t < m; ++t) {
      if (colsum[t] > n1) { n1 = colsum[t]; js = t; }
      if (rowsum[t] > ninf) { ninf = rowsum[t]; is = t; }
    }
    hdr->n1 = n1; hdr->ninf = ninf; hdr->jstar = js; hdr->istar = is;
    hdr->auto_alpha = !(alpha_in > 0.f);
    hdr->alpha = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * ninf);
    hdr->pad0 = hdr->pad1 = 0;
  }
  __syncthreads();
}

// Forward iteration.  smem: three matrices (W, X, P), 3 * NsTile<MP>::mat_bytes.  Xh (global, [T+1][m][m])
// receives X_0 .. X_T in fp32.
template <int MP>
__device__ void ns_forward_smem(int m, int T, float eps, float alpha_in, const float* W, float* Xh, NsHdr* hdr,
                                bf16* smem, float* red) {
  using TL = NsTile<MP>;
  bf16* sW = smem; bf16* sX = smem + 2 * TL::MAT; bf16* sP = smem + 4 * TL::MAT;
  const long long mm = (long long)m * m;
  ns_norms(m, eps, alpha_in, W, hdr, red);
  const float alpha = hdr->alpha;
  global_to_smem<MP>(W, m, eps, 1.f, false, sW);
  global_to_smem<MP>(W, m, eps, alpha, true, sX);                       // X_0 = alpha (W + eps I)^T
  for (long long e = threadIdx.x; e < mm; e += 256) {
    const int i = (int)(e / m), j = (int)(e % m);
    Xh[e] = alpha * (W[(long long)j * m + i] + (i == j ? eps : 0.f));
  }
  __syncthreads();
  float acc[TL::MT][TL::NT][4];
  for (int k = 0; k < T; ++k) {
    smem_gemm<MP, false, false>(acc, sW, sX, false);                    // W X_k
#pragma unroll
    for (int a = 0; a < TL::MT; ++a)
#pragma unroll
      for (int t = 0; t < TL::NT; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          acc[a][t][q] = ((i == j && i < m) ? 2.f : 0.f) - acc[a][t][q];   // 2I - W X_k
        }
    frag_to_smem<MP>(acc, sP);
    __syncthreads();
    smem_gemm<MP, false, false>(acc, sX, sP, false);                    // X_{k+1} = X_k (2I - W X_k)
    frag_to_global<MP>(acc, Xh + (long long)(k + 1) * mm, m);
    __syncthreads();                                                    // every warp is done reading X_k
    frag_to_smem<MP>(acc, sX);
    __syncthreads();
  }
}

// Adjoint.  smem: five matrices (W, A, G, P, H).  Xh: fp32 history from the forward pass; G0 = dLoss/dX_T
// (global fp32).  Writes dW (global fp32 [m][m]); Gt is a global fp32 [m][m] scratch.
template <int MP>
__device__ void ns_backward_smem(int m, int T, float eps, const float* W, const float* Xh, const NsHdr* hdr,
                                 const float* G0, float* dW, float* Gt, bf16* smem, float* red) {
  using TL = NsTile<MP>;
  bf16* sW = smem; bf16* sA = smem + 2 * TL::MAT; bf16* sG = smem + 4 * TL::MAT;
  bf16* sP = smem + 6 * TL::MAT; bf16* sH = smem + 8 * TL::MAT;
  const long long mm = (long long)m * m;
  float G[TL::MT][TL::NT][4], dWr[TL::MT][TL::NT][4], acc[TL::MT][TL::NT][4];
  global_to_smem<MP>(W, m, eps, 1.f, false, sW);
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int i, j;
        frag_ij<MP>(a, t, q, i, j);
        G[a][t][q] = (i < m && j < m) ? G0[(long long)i * m + j] : 0.f;
        dWr[a][t][q] = 0.f;
      }
  frag_to_smem<MP>(G, sG);
  for (int k = T - 1; k >= 0; --k) {
    __syncthreads();                                                    // previous readers of sA, sG writers done
    global_to_smem<MP>(Xh + (long long)k * mm, m, 0.f, 1.f, false, sA);  // A = X_k
    __syncthreads();
    smem_gemm<MP, true, false>(acc, sA, sG, false);                     // H = A^T G
    frag_to_smem<MP>(acc, sH);
    smem_gemm<MP, false, false>(acc, sW, sA, false);                    // P = W A
    frag_to_smem<MP>(acc, sP);
    __syncthreads();
    smem_gemm<MP, false, true>(acc, sH, sA, false);                     // H A^T
#pragma unroll
    for (int a = 0; a < TL::MT; ++a)
#pragma unroll
      for (int t = 0; t < TL::NT; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) dWr[a][t][q] -= acc[a][t][q];       // dW -= H A^T
    smem_gemm<MP, false, true>(acc, sG, sP, false);                     // G P^T
    smem_gemm<MP, true, false>(acc, sW, sH, true);                      // + W^T H
#pragma unroll
    for (int a = 0; a < TL::MT; ++a)
#pragma unroll
      for (int t = 0; t < TL::NT; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) G[a][t][q] = 2.f * G[a][t][q] - acc[a][t][q];
    __syncthreads();                                                    // every warp is done reading sG
    frag_to_smem<MP>(G, sG);
  }
  // X_0 = alpha (W + eps I)^T:  d alpha = <G, W^T>,  dW += alpha G^T, then the alpha(W) terms
  const float alpha = hdr->alpha;
  float part = 0.f;
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int i, j;
        frag_ij<MP>(a, t, q, i, j);
        if (i < m && j < m) part += G[a][t][q] * (W[(long long)j * m + i] + (i == j ? eps : 0.f));
      }
  frag_to_global<MP>(G, Gt, m);
  const float dalpha = block_sum(part, red);                            // contains __syncthreads: Gt is visible
  const bool aa = hdr->auto_alpha != 0;
  const int js = hdr->jstar, is = hdr->istar;
  const float c1 = dalpha * (-alpha / hdr->n1), c2 = dalpha * (-alpha / hdr->ninf);
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int i, j;
        frag_ij<MP>(a, t, q, i, j);
        if (i < m && j < m) {
          float v = dWr[a][t][q] + alpha * Gt[(long long)j * m + i];
          if (aa) {
            const float w = W[(long long)i * m + j] + (i == j ? eps : 0.f);
            const float sg = w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f);
            if (j == js) v += c1 * sg;
            if (i == is) v += c2 * sg;
          }
          dW[(long long)i * m + j] = v;
        }
      }
  __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Adjoint for 64 < m <= 128.  Five hi/lo matrices of 128 x 128 do not fit in one SM's shared
// memory, so three stay resident (A = X_k, G, and H which is later reused for P) while W, which
// only ever appears as the left operand (W A and W^T H), is streamed from global memory (L2) in
// K-chunks of 32 through a small staging buffer.  G and dW are kept in fp32 in global memory and
// touched fragment-wise (each thread reads and writes only its own elements).
// smem: 3 * NsTile<128>::mat_bytes + kStage128Bytes.
// ---------------------------------------------------------------------------------------------
constexpr int kStageEl = 128 * 40;                                    // bf16 elements of one staged part (hi or lo)
constexpr size_t kStage128Bytes = (size_t)2 * kStageEl * sizeof(bf16);

// acc (+)= op(W + eps I) B, W [m][m] in global memory, B resident ([K][N], hi/lo); TRA: op = transpose
template <bool TRA>
__device__ void smem_gemm_stream_w(float (&acc)[2][8][4], const float* W, int m, float eps, bf16* stage, const bf16* Bm,
                                   bool accumulate) {
  using TL = NsTile<128>;
  const int tid = threadIdx.x, wm = TL::wm(), wn = TL::wn();
  if (!accumulate) {
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[a][t][q] = 0.f;
  }
  // row-chunk form (TRA = false): stage[128][40], thread -> (row tid/2, 16 cols); chunk = W[:, k0..k0+31]
  // col-chunk form (TRA = true) : stage[32][136], thread -> (row tid/8, 16 cols); chunk = W[k0..k0+31, :]
  const int r = TRA ? (tid >> 3) : (tid >> 1), cb = TRA ? (tid & 7) * 16 : (tid & 1) * 16;
  constexpr int LDS_ = TRA ? 136 : 40;
  float v[16];
  auto fetch = [&](int k0) {
    const int gr = TRA ? k0 + r : r, gc = TRA ? cb : k0 + cb;
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const int cc = gc + q;
      float x = (gr < m && cc < m) ? W[(long long)gr * m + cc] : 0.f;
      if (gr == cc && gr < m) x += eps;
      v[q] = x;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < 128; k0 += 32) {
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 16; q += 4) {
      uint2 h, l;
      split4(make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]), h, l);
      *reinterpret_cast<uint2*>(stage + r * LDS_ + cb + q) = h;
      *reinterpret_cast<uint2*>(stage + kStageEl + r * LDS_ + cb + q) = l;
    }
    __syncthreads();
    if (k0 + 32 < 128) fetch(k0 + 32);
#pragma unroll
    for (int kk = 0; kk < 32; kk += 16) {
      uint32_t ah[2][4], al[2][4];
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        if (TRA) { ldsm_x4_t(ah[a], addr_at(stage, 136, kk, wm + a * 16)); ldsm_x4_t(al[a], addr_at(stage + kStageEl, 136, kk, wm + a * 16)); }
        else     { ldsm_x4(ah[a], addr_a(stage, 40, wm + a * 16, kk));     ldsm_x4(al[a], addr_a(stage + kStageEl, 40, wm + a * 16, kk)); }
      }
      uint32_t bh4[4][4], bl4[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        ldsm_x4_t(bh4[t], addr_bt(Bm, TL::LD, k0 + kk, wn + t * 16));
        ldsm_x4_t(bl4[t], addr_bt(Bm + TL::MAT, TL::LD, k0 + kk, wn + t * 16));
      }
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          mma_bf16(acc[a][2 * t], al[a], bh4[t][0], bh4[t][1]);
          mma_bf16(acc[a][2 * t + 1], al[a], bh4[t][2], bh4[t][3]);
        }
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          mma_bf16(acc[a][2 * t], ah[a], bl4[t][0], bl4[t][1]);
          mma_bf16(acc[a][2 * t + 1], ah[a], bl4[t][2], bl4[t][3]);
        }
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          mma_bf16(acc[a][2 * t], ah[a], bh4[t][0], bh4[t][1]);
          mma_bf16(acc[a][2 * t + 1], ah[a], bh4[t][2], bh4[t][3]);
        }
    }
  }
  __syncthreads();
}

// Gf, T1: global fp32 [m][m] scratch.  dW: output (global fp32 [m][m]).
__device__ void ns_backward_smem128(int m, int T, float eps, const float* W, const float* Xh, const NsHdr* hdr,
                                    const float* G0, float* dW, float* Gf, float* T1, bf16* smem, float* red) {
  using TL = NsTile<128>;
  constexpr int MP = 128;
  bf16* sA = smem; bf16* sG = smem + 2 * TL::MAT; bf16* sH = smem + 4 * TL::MAT; bf16* stage = smem + 6 * TL::MAT;
  const long long mm = (long long)m * m;
  float acc[2][8][4];
  for (long long e = threadIdx.x; e < mm; e += 256) { Gf[e] = G0[e]; dW[e] = 0.f; }
  global_to_smem<MP>(G0, m, 0.f, 1.f, false, sG);
  for (int k = T - 1; k >= 0; --k) {
    __syncthreads();
    global_to_smem<MP>(Xh + (long long)k * mm, m, 0.f, 1.f, false, sA);     // A = X_k
    __syncthreads();
    smem_gemm<MP, true, false>(acc, sA, sG, false);                        // H = A^T G
    frag_to_smem<MP>(acc, sH);
    __syncthreads();
    smem_gemm<MP, false, true>(acc, sH, sA, false);                        // H A^T
    // dW -= H A^T on this thread's own elements; all loads of a tile row are issued before the stores
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      float old[8][4];
#pragma unroll
      for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          old[t][q] = (i < m && j < m) ? dW[(long long)i * m + j] : 0.f;
        }
#pragma unroll
      for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          if (i < m && j < m) dW[(long long)i * m + j] = old[t][q] - acc[a][t][q];
        }
    }
    smem_gemm_stream_w<true>(acc, W, m, eps, stage, sH, false);             // W^T H
    frag_to_global<MP>(acc, T1, m);
    smem_gemm_stream_w<false>(acc, W, m, eps, stage, sA, false);            // P = W A
    frag_to_smem<MP>(acc, sH);                                             // H is dead: its buffer takes P
    __syncthreads();
    smem_gemm<MP, false, true>(acc, sG, sH, false);                        // G P^T
    __syncthreads();                                                       // every warp is done reading sG
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      float g0[8][4], t1[8][4];
#pragma unroll
      for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          const bool in = i < m && j < m;
          g0[t][q] = in ? Gf[(long long)i * m + j] : 0.f;
          t1[t][q] = in ? T1[(long long)i * m + j] : 0.f;
        }
#pragma unroll
      for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          const float gn = 2.f * g0[t][q] - acc[a][t][q] - t1[t][q];   // 2G - G P^T - W^T H
          if (i < m && j < m) Gf[(long long)i * m + j] = gn;
          acc[a][t][q] = (i < m && j < m) ? gn : 0.f;
        }
    }
    frag_to_smem<MP>(acc, sG);
  }
  __syncthreads();
  // acc holds G in fragment layout when T > 0; reload it so that T = 0 works too
  const float alpha = hdr->alpha;
  float part = 0.f;
  for (long long e = threadIdx.x; e < mm; e += 256) {
    const int i = (int)(e / m), j = (int)(e % m);
    part += Gf[e] * (W[(long long)j * m + i] + (i == j ? eps : 0.f));
  }
  const float dalpha = block_sum(part, red);
  const bool aa = hdr->auto_alpha != 0;
  const int js = hdr->jstar, is = hdr->istar;
  const float c1 = dalpha * (-alpha / hdr->n1), c2 = dalpha * (-alpha / hdr->ninf);
  for (long long e = threadIdx.x; e < mm; e += 256) {
    const int i = (int)(e / m), j = (int)(e % m);
    float v = dW[e] + alpha * Gf[(long long)j * m + i];
    if (aa) {
      const float w = W[e] + (i == j ? eps : 0.f);
      const float sg = w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f);
      if (j == js) v += c1 * sg;
      if (i == is) v += c2 * sg;
    }
    dW[e] = v;
  }
  __syncthreads();
}

}  // namespace ln
