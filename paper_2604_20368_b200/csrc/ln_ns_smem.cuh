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
#pragma unroll 2
  for (int k0 = 0; k0 < MP; k0 += 16) {
    uint32_t ah[MT][4], al[MT][4];
#pragma unroll
    for (int a = 0; a < MT; ++a) {
      if (TRA) { ldsm_x4_t(ah[a], addr_at(A, LD, k0, wm + a * 16)); ldsm_x4_t(al[a], addr_at(A + MAT, LD, k0, wm + a * 16)); }
      else     { ldsm_x4(ah[a], addr_a(A, LD, wm + a * 16, k0));    ldsm_x4(al[a], addr_a(A + MAT, LD, wm + a * 16, k0)); }
    }
#pragma unroll
    for (int t = 0; t < NT; t += 2) {
      uint32_t bh4[4], bl4[4];
      if (TRB) { ldsm_x4(bh4, addr_b(Bm, LD, wn + t * 8, k0));    ldsm_x4(bl4, addr_b(Bm + MAT, LD, wn + t * 8, k0)); }
      else     { ldsm_x4_t(bh4, addr_bt(Bm, LD, k0, wn + t * 8)); ldsm_x4_t(bl4, addr_bt(Bm + MAT, LD, k0, wn + t * 8)); }
#pragma unroll
      for (int a = 0; a < MT; ++a) {
        mma_bf16(acc[a][t], al[a], bh4[0], bh4[1]);
        mma_bf16(acc[a][t], ah[a], bl4[0], bl4[1]);
        mma_bf16(acc[a][t], ah[a], bh4[0], bh4[1]);
        mma_bf16(acc[a][t + 1], al[a], bh4[2], bh4[3]);
        mma_bf16(acc[a][t + 1], ah[a], bl4[2], bl4[3]);
        mma_bf16(acc[a][t + 1], ah[a], bh4[2], bh4[3]);
      }
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

// global fp32 [m][m] (+ diag on the diagonal, times scale, optionally transposed) -> shared hi/lo, zero padded
template <int MP>
__device__ __forceinline__ void global_to_smem(const float* src, int m, float diag, float scale, bool transpose, bf16* dst) {
  using TL = NsTile<MP>;
  for (int e = threadIdx.x; e < MP * MP; e += 256) {
    const int i = e / MP, j = e % MP;
    float v = 0.f;
    if (i < m && j < m) {
      v = transpose ? src[(long long)j * m + i] : src[(long long)i * m + j];
      if (i == j) v += diag;
      v *= scale;
    }
    bf16 h, l;
    split2(v, h, l);
    dst[i * TL::LD + j] = h;
    dst[TL::MAT + i * TL::LD + j] = l;
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

}  // namespace ln
