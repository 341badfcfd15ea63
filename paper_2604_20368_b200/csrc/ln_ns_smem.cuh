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
__device__ __forceinline__ void frag_to_global(const float (&acc)[NsTile<MP>::MT][NsTile<MP>::NT][4], float* dst, int m, int ld) {
  using TL = NsTile<MP>;
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        int i, j;
        frag_ij<MP>(a, t, q, i, j);
        if (i < m && j < m) dst[(long long)i * ld + j] = acc[a][t][q];
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


// One matrix of this path as it lies in shared memory (hi part, lo part, rows of NsTile<MP>::LD bf16) is also
// the format of the iterate history in global memory: the forward pass copies its operand images out, the
// backward pass copies them back in with cp.async, and nothing is split or converted twice.
template <int MP> __device__ __forceinline__ void image_to_global(const bf16* src, float* dst) {
  constexpr int CH = (int)(NsTile<MP>::mat_bytes / 16);
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  for (int c = threadIdx.x; c < CH; c += 256) d4[c] = s4[c];
}
// asynchronous global -> shared copy of one image; every thread commits exactly one group per call
template <int MP> __device__ __forceinline__ void image_prefetch(const float* src, bf16* dst, bool issue) {
  constexpr int CH = (int)(NsTile<MP>::mat_bytes / 16);
  if (issue) {
    const char* g = reinterpret_cast<const char*>(src);
    const uint32_t s0 = smem_u32(dst);
    for (int c = threadIdx.x; c < CH; c += 256)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s0 + 16u * c), "l"(g + 16ll * c) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}
// all but the most recent group of this thread have landed
__device__ __forceinline__ void image_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// Forward iteration.  smem: three matrices (W, X, P), 3 * NsTile<MP>::mat_bytes.  Histories in global memory,
// slots of hs floats: Xh slot k < T receives the operand image of X_k, slot T receives X_T in fp32 (leading
// dimension ld >= m); Ph slot k (may be NULL) receives the image of Q_k = 2I - W X_k.
template <int MP>
__device__ void ns_forward_smem(int m, int T, float eps, float alpha_in, const float* W, float* Xh, float* Ph, int ld,
                                long long hs, NsHdr* hdr, bf16* smem, float* red, float& bad) {
  // bad: this thread's count of non-finite entries of X_T (from its registers: nothing is read back)
  using TL = NsTile<MP>;
  bf16* sW = smem; bf16* sX = smem + 2 * TL::MAT; bf16* sP = smem + 4 * TL::MAT;
  // W + eps I is first staged in fp32 (in the space of P, which is not needed yet): norms, the split
  // copy of W, X_0 = alpha W^T and its fp32 copy for the backward pass are all built from there, so
  // global memory is read exactly once, coalesced.
  float* Wf = reinterpret_cast<float*>(sP);
  constexpr int PF = MP + 4;
  constexpr int PER = MP * MP / 256;
#pragma unroll 1
  for (int b0 = 0; b0 < PER; b0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = (b0 + u) * 256 + threadIdx.x, i = e / MP, j = e % MP;
      v[u] = (i < m && j < m) ? W[(long long)i * m + j] + (i == j ? eps : 0.f) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = (b0 + u) * 256 + threadIdx.x, i = e / MP, j = e % MP;
      Wf[i * PF + j] = v[u];
    }
  }
  __syncthreads();
  {
    float* colsum = red; float* rowsum = red + 256;
    const int t = threadIdx.x;
    if (t < m) {
      float cs = 0.f, rs = 0.f;
      for (int i = 0; i < m; ++i) { cs += fabsf(Wf[i * PF + t]); rs += fabsf(Wf[t * PF + i]); }
      colsum[t] = cs; rowsum[t] = rs;
    }
    __syncthreads();
    if (t == 0) {
      float n1 = -1.f, ninf = -1.f; int js = 0, is = 0;
      for (int q = 0; q < m; ++q) {                 // strict > keeps the lowest index on ties
        if (colsum[q] > n1) { n1 = colsum[q]; js = q; }
        if (rowsum[q] > ninf) { ninf = rowsum[q]; is = q; }
      }
      hdr->n1 = n1; hdr->ninf = ninf; hdr->jstar = js; hdr->istar = is;
      hdr->auto_alpha = !(alpha_in > 0.f);
      hdr->alpha = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * ninf);
      hdr->pad0 = hdr->pad1 = 0;
    }
    __syncthreads();
  }
  const float alpha = hdr->alpha;
  for (int e = threadIdx.x; e < MP * MP; e += 256) {
    const int i = e / MP, j = e % MP;
    bf16 h, l;
    split2(Wf[i * PF + j], h, l);
    sW[i * TL::LD + j] = h; sW[TL::MAT + i * TL::LD + j] = l;
    const float x0 = alpha * Wf[j * PF + i];                          // X_0 = alpha (W + eps I)^T
    split2(x0, h, l);
    sX[i * TL::LD + j] = h; sX[TL::MAT + i * TL::LD + j] = l;
    if (T == 0 && i < m && j < m) { Xh[(long long)i * ld + j] = x0; bad += isfinite(x0) ? 0.f : 1.f; }
  }
  __syncthreads();
  if (T > 0) image_to_global<MP>(sX, Xh);
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
    if (Ph) image_to_global<MP>(sP, Ph + k * hs);                       // kept for the backward pass
    smem_gemm<MP, false, false>(acc, sX, sP, false);                    // X_{k+1} = X_k (2I - W X_k)
    if (k + 1 == T) {
      frag_to_global<MP>(acc, Xh + T * hs, m, ld);
#pragma unroll
      for (int a = 0; a < TL::MT; ++a)
#pragma unroll
        for (int t = 0; t < TL::NT; ++t)
#pragma unroll
          for (int q = 0; q < 4; ++q) bad += isfinite(acc[a][t][q]) ? 0.f : 1.f;      // padding is zero, hence finite
    }
    __syncthreads();                                                    // every warp is done reading X_k
    frag_to_smem<MP>(acc, sX);
    __syncthreads();
    if (k + 1 < T) image_to_global<MP>(sX, Xh + (k + 1) * hs);
  }
}

// global fp32 [m][m] with leading dimension ld -> shared hi/lo, with 128-bit loads when ld allows it
// (columns >= m of a padded row hold nothing defined and are masked to zero)
template <int MP>
__device__ __forceinline__ void global_to_smem_fast(const float* __restrict__ src, int m, int ld, bf16* dst) {
  using TL = NsTile<MP>;
  if ((ld & 3) == 0) {
    constexpr int PER4 = MP * MP / 4 / 256;       // float4 pieces per thread
#pragma unroll 1
    for (int b0 = 0; b0 < PER4; b0 += 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = ((b0 + u) * 256 + threadIdx.x) * 4, i = e / MP, j = e % MP;
        v[u] = (b0 + u < PER4 && i < m && j < m) ? *reinterpret_cast<const float4*>(src + (long long)i * ld + j)
                                                 : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (b0 + u >= PER4) break;
        const int e = ((b0 + u) * 256 + threadIdx.x) * 4, i = e / MP, j = e % MP;
        float4 x = v[u];
        if (j + 1 >= m) x.y = 0.f;
        if (j + 2 >= m) x.z = 0.f;
        if (j + 3 >= m) x.w = 0.f;
        uint2 h, l;
        split4(x, h, l);
        *reinterpret_cast<uint2*>(dst + i * TL::LD + j) = h;
        *reinterpret_cast<uint2*>(dst + TL::MAT + i * TL::LD + j) = l;
      }
    }
  } else {
    for (int e = threadIdx.x; e < MP * MP; e += 256) {
      const int i = e / MP, j = e % MP;
      bf16 h, l;
      split2((i < m && j < m) ? src[(long long)i * ld + j] : 0.f, h, l);
      dst[i * TL::LD + j] = h;
      dst[TL::MAT + i * TL::LD + j] = l;
    }
  }
}

// End of the adjoint, shared by the shared-memory and tcgen05 paths.  On entry dW holds minus the
// accumulated sum of H A^T and Gf the final G (both global fp32, leading dimension ld).
__device__ inline void ns_backward_tail(int m, float eps, const float* W, int ld, const NsHdr* hdr, float* dW, const float* Gf,
                                        float* red) {
  // X_0 = alpha (W + eps I)^T:  d alpha = <G, W^T>,  dW += alpha G^T, then the alpha(W) terms
  const float alpha = hdr->alpha;
  float part = 0.f;
  const int mlog = m * m;
  for (int e = threadIdx.x; e < mlog; e += 256) {
    const int i = e / m, j = e % m;
    part += Gf[(long long)i * ld + j] * (W[(long long)j * m + i] + (i == j ? eps : 0.f));
  }
  const float dalpha = block_sum(part, red);
  const bool aa = hdr->auto_alpha != 0;
  const int js = hdr->jstar, is = hdr->istar;
  const float c1 = dalpha * (-alpha / hdr->n1), c2 = dalpha * (-alpha / hdr->ninf);
  for (int e0 = threadIdx.x; e0 < mlog; e0 += 1024) {
    float d0[4], gt[4], w0[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * 256, i = e / m, j = e % m;
      const bool in = e < mlog;
      d0[u] = in ? dW[(long long)i * ld + j] : 0.f; gt[u] = in ? Gf[(long long)j * ld + i] : 0.f; w0[u] = in ? W[e] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u * 256;
      if (e >= mlog) break;
      const int i = e / m, j = e % m;
      float v = d0[u] + alpha * gt[u];
      if (aa) {
        const float w = w0[u] + (i == j ? eps : 0.f);
        const float sg = w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f);
        if (j == js) v += c1 * sg;
        if (i == is) v += c2 * sg;
      }
      dW[(long long)i * ld + j] = v;
    }
  }
  __syncthreads();
}

// Adjoint of the iteration for a symmetric W (the landmark kernel matrix is symmetric bit for bit).
// Per step k (A = X_k, Q = 2I - W A, both saved as operand images by the forward pass):
//     H = A^T G,   dW -= H A^T,   G <- G Q^T + Q^T G - 2G.
// In general the last term of the step adjoint is W^T H = (A W)^T G; for symmetric W every iterate is a
// polynomial in W, so A W = W A up to rounding, (A W)^T G = (2I - Q)^T G, and W itself is not needed inside
// the loop.  Four matrices are resident in shared memory (A, Q, G, H: 4 * NsTile<MP>::mat_bytes); A and Q of
// the next step arrive by cp.async while this step computes.  G is kept in fp32 in registers (accumulator
// layout) and re-split into shared memory after each update.
// Xh, Ph: history slots of hs floats; G0 = dLoss/dX_T (fp32, leading dimension ld); Gf: global fp32 [m][ld]
// scratch that receives the final G for the tail.
template <int MP>
__device__ void ns_backward_smem(int m, int T, float eps, const float* W, const float* Xh, const float* Ph, int ld,
                                 long long hs, const NsHdr* hdr, const float* G0, float* dW, float* Gf, bf16* smem,
                                 float* red) {
  using TL = NsTile<MP>;
  bf16* sA = smem; bf16* sQ = smem + 2 * TL::MAT; bf16* sG = smem + 4 * TL::MAT; bf16* sH = smem + 6 * TL::MAT;
  image_prefetch<MP>(Xh + (long long)(T - 1) * hs, sA, T > 0);
  image_prefetch<MP>(Ph + (long long)(T - 1) * hs, sQ, T > 0);
  float acc[TL::MT][TL::NT][4], dWr[TL::MT][TL::NT][4], Gr[TL::MT][TL::NT][4];
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        int i, j;
        frag_ij<MP>(a, t, 2 * h, i, j);                                    // j is even: (j, j+1) are this thread's
        float2 g = make_float2(0.f, 0.f);
        if (i < m && j + 1 < m && (ld & 1) == 0) g = *reinterpret_cast<const float2*>(G0 + (long long)i * ld + j);
        else {
          if (i < m && j < m) g.x = G0[(long long)i * ld + j];
          if (i < m && j + 1 < m) g.y = G0[(long long)i * ld + j + 1];
        }
        Gr[a][t][2 * h] = g.x; Gr[a][t][2 * h + 1] = g.y;
        dWr[a][t][2 * h] = 0.f; dWr[a][t][2 * h + 1] = 0.f;
      }
  frag_to_smem<MP>(Gr, sG);
  for (int k = T - 1; k >= 0; --k) {
    image_wait_all_but_one();                                              // A = X_k has landed (Q_k may be in flight)
    __syncthreads();
    smem_gemm<MP, true, false>(acc, sA, sG, false);                        // H = A^T G
    frag_to_smem<MP>(acc, sH);
    __syncthreads();
    smem_gemm<MP, false, true>(dWr, sH, sA, true);                         // accumulates H A^T (dW = -sum)
    __syncthreads();                                                       // every warp is done reading A
    image_prefetch<MP>(Xh + (long long)(k - 1) * hs, sA, k > 0);
    image_wait_all_but_one();                                              // Q_k has landed
    __syncthreads();
    smem_gemm<MP, false, true>(acc, sG, sQ, false);                        // G Q^T
    smem_gemm<MP, true, false>(acc, sQ, sG, true);                         // + Q^T G
    __syncthreads();                                                       // every warp is done reading G and Q
    image_prefetch<MP>(Ph + (long long)(k - 1) * hs, sQ, k > 0);
#pragma unroll
    for (int a = 0; a < TL::MT; ++a)
#pragma unroll
      for (int t = 0; t < TL::NT; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          int i, j;
          frag_ij<MP>(a, t, q, i, j);
          Gr[a][t][q] = (i < m && j < m) ? acc[a][t][q] - 2.f * Gr[a][t][q] : 0.f;
        }
    frag_to_smem<MP>(Gr, sG);
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
  for (int a = 0; a < TL::MT; ++a)
#pragma unroll
    for (int t = 0; t < TL::NT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) dWr[a][t][q] = -dWr[a][t][q];
  frag_to_global<MP>(dWr, dW, m, ld);
  frag_to_global<MP>(Gr, Gf, m, ld);
  __syncthreads();
  ns_backward_tail(m, eps, W, ld, hdr, dW, Gf, red);
  __syncthreads();
}

}  // namespace ln
