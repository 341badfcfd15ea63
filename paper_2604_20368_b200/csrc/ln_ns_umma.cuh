// Newton-Schulz (Alg. 2) and its adjoint for m <= 128 on the 5th-generation tensor cores:
// tcgen05.mma issued by one thread, operands as bf16 hi + lo images in shared memory (three MMAs
// per product: lo*hi, hi*lo, hi*hi), fp32 accumulators in tensor memory (TMEM), read back with
// tcgen05.ld for the epilogue that produces the next operand image.  One CTA of 256 threads per head;
// the iterate never leaves the SM except for the history the backward pass needs.
//
// Two sizes, UM = 128 (64 < m <= 128) and UM = 64 (m <= 64), the matrix padded with zeros to UM x UM.
// UM = 128: thread t owns row 32 (warp % 4) + lane of the accumulator and the column half warp / 4 (64 values).
// UM = 64 : an M = 64 accumulator keeps row r in TMEM lane 32 (r / 16) + r % 16, so the first 16 lanes of every warp
//           own row 16 (warp % 4) + lane and the column half warp / 4 (32 values); the other lanes only take part
//           in the warp-wide TMEM loads and the barriers.
#pragma once
#include "ln_mma.cuh"
#include "ln_umma.cuh"

namespace ln {

// geometry of one size: UIMG = bf16 elements of one image part (hi or lo), NV = values a thread owns of its row
template <int UM> struct UmmaGeo {
  static constexpr int UIMG = UM * UM;
  static constexpr size_t mat_bytes = (size_t)2 * UIMG * sizeof(bf16);     // hi + lo: 64 KiB (UM = 128), 16 KiB (UM = 64)
  static constexpr int NV = UM / 2;
  static constexpr int LOG = UM == 128 ? 7 : 6;
  __device__ static __forceinline__ bool active() { return UM == 128 || (threadIdx.x & 31) < 16; }
  __device__ static __forceinline__ int row() {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    return UM == 128 ? (warp & 3) * 32 + lane : (warp & 3) * 16 + (lane & 15);
  }
  __device__ static __forceinline__ int col0() { return (int)(threadIdx.x >> 7) * NV; }
};
constexpr size_t kUmmaMatBytes = UmmaGeo<128>::mat_bytes;
constexpr size_t kUmmaMatBytes64 = UmmaGeo<64>::mat_bytes;

struct UmmaCtl {                              // small static shared state of the tcgen05 kernels
  unsigned long long mbar;                    // completion of MMAs
  unsigned long long mbar_ld;                 // arrival of a bulk-copied operand image
  uint32_t tmem_base;
  int timeout;
};

// D[tmem_col .. +128) (+)= op(A) op(B) with split operands (hi at image, lo at image + UIMG); one thread.
//   a_k: A image rows are M (A = X) else rows are K (A = X^T);  b_k: B image rows are N (B = X^T) else rows are K (B = X)
template <int UM>
__device__ __forceinline__ void umma_gemm(uint32_t tmem_d, const bf16* A, bool a_k, const bf16* Bm, bool b_k, bool accumulate) {
  constexpr int UIMG = UmmaGeo<UM>::UIMG;
  const uint32_t idesc = umma::instr_desc(UM, !a_k, !b_k, UM);
  bool acc = accumulate;
#pragma unroll 1
  for (int part = 0; part < 3; ++part) {      // lo*hi, hi*lo, hi*hi
    const bf16* a = A + (part == 0 ? UIMG : 0);
    const bf16* b = Bm + (part == 1 ? UIMG : 0);
#pragma unroll
    for (int ks = 0; ks < UM / 16; ++ks) {
      umma::mma(tmem_d, umma::operand_desc(a, UM, a_k, ks), umma::operand_desc(b, UM, b_k, ks), idesc, acc);
      acc = true;
    }
  }
}

// issue (thread 0) + wait (everyone); returns false on a timed-out wait
// `phase` is each thread's own copy of the mbarrier phase (identical in all threads)
// drain_stores: thread 0 first lets its bulk stores finish reading shared memory, so that when the barrier
// completes the buffers those stores read may be overwritten by everybody
template <int UM>
__device__ __forceinline__ bool umma_run(UmmaCtl& ctl, uint32_t& phase, uint32_t tmem_d, const bf16* A, bool a_k, const bf16* Bm,
                                         bool b_k, bool accumulate, const bf16* A2 = nullptr, bool a2_k = true,
                                         const bf16* B2 = nullptr, bool b2_k = true, bool drain_stores = false) {
  if (threadIdx.x == 0) {
    umma::fence_after_sync();
    umma_gemm<UM>(tmem_d, A, a_k, Bm, b_k, accumulate);
    if (A2) umma_gemm<UM>(tmem_d, A2, a2_k, B2, b2_k, true);
    if (drain_stores) umma::bulk_store_wait_read();
    umma::commit(&ctl.mbar);
  }
  const bool ok = umma::mbar_wait(&ctl.mbar, phase & 1);
  phase ^= 1u;
  umma::fence_after_sync();
  return ok;
}

// NV consecutive columns (this thread's half) of its accumulator row (every lane of the warp takes part in the load)
template <int NV>
__device__ __forceinline__ void umma_row(uint32_t tmem_base, int col0, float (&v)[NV]) {
#pragma unroll
  for (int c = 0; c < NV; c += 32) {
    float a[32];
    umma::tmem_ld32(umma::tmem_addr(tmem_base, col0 + c), a);
#pragma unroll
    for (int q = 0; q < 32; ++q) v[c + q] = a[q];
  }
}

// this thread's 64 values of row i -> global fp32 row (leading dimension ld, a multiple of 4): 128-bit stores.
// Columns in [m, ld) receive whatever the accumulator holds there (zero); readers mask them anyway.
template <int NV>
__device__ __forceinline__ void umma_row_to_global(const float (&v)[NV], float* dst_row, int j0, int ld) {
#pragma unroll
  for (int p = 0; p < NV / 4; ++p) {
    const int c = j0 + 4 * p;
    if (c < ld) *reinterpret_cast<float4*>(dst_row + c) = make_float4(v[4 * p], v[4 * p + 1], v[4 * p + 2], v[4 * p + 3]);
  }
}

// this thread's NV values of row i -> the hi/lo image of a UM x UM matrix (16-byte pieces)
template <int UM>
__device__ __forceinline__ void umma_row_to_image(const float (&v)[UM / 2], int i, int j0, bf16* image) {
  constexpr int UIMG = UmmaGeo<UM>::UIMG;
#pragma unroll
  for (int p = 0; p < UM / 16; ++p) {
    uint2 h0, l0, h1, l1;
    split4(make_float4(v[8 * p], v[8 * p + 1], v[8 * p + 2], v[8 * p + 3]), h0, l0);
    split4(make_float4(v[8 * p + 4], v[8 * p + 5], v[8 * p + 6], v[8 * p + 7]), h1, l1);
    const int off = umma::img(i, j0 + 8 * p, UM);
    *reinterpret_cast<uint4*>(image + off) = make_uint4(h0.x, h0.y, h1.x, h1.y);
    *reinterpret_cast<uint4*>(image + UIMG + off) = make_uint4(l0.x, l0.y, l1.x, l1.y);
  }
}

__device__ __forceinline__ void umma_begin(UmmaCtl& ctl, int ncols) {
  if (threadIdx.x == 0) { umma::mbar_init(&ctl.mbar, 1); umma::mbar_init(&ctl.mbar_ld, 1); ctl.timeout = 0; }
  if ((threadIdx.x >> 5) == 0) umma::tmem_alloc(&ctl.tmem_base, ncols);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
}
__device__ __forceinline__ void umma_end(UmmaCtl& ctl, int ncols) {
  umma::fence_before_sync();
  __syncthreads();
  if ((threadIdx.x >> 5) == 0) umma::tmem_dealloc(ctl.tmem_base, ncols);
}
// end of a step: what the threads wrote to shared memory becomes visible to the tensor core, and
// their TMEM reads are ordered before the next MMA that overwrites the accumulator
__device__ __forceinline__ void umma_step_done(UmmaCtl& ctl, bool ok) {
  if (!ok) ctl.timeout = 1;
  umma::fence_smem_to_mma();
  umma::fence_before_sync();
  __syncthreads();
}


// Forward iteration.  smem: images W, X, Q (3 * mat_bytes).  Histories in global memory, slots of hs floats
// (hs * 4 >= mat_bytes): Xh slot k < T receives the operand image of X_k, slot T receives X_T in fp32 (leading
// dimension ld); Ph slot k (may be NULL) receives the image of Q_k = 2I - W X_k.  The images leave by bulk copies
// that one thread issues and that run beside the next product.  Returns false if a tensor-core wait timed out.
template <int UM>
__device__ bool ns_forward_umma(int m, int T, float eps, float alpha_in, const float* W, float* Xh, float* Ph, int ld,
                                long long hs, NsHdr* hdr, bf16* smem, float* red, UmmaCtl& ctl, float& bad) {
  // bad: this thread's count of non-finite entries of X_T (from its registers)
  typedef UmmaGeo<UM> Geo;
  constexpr int UIMG = Geo::UIMG, NV = Geo::NV, LOG = Geo::LOG;
  constexpr uint32_t MATB = (uint32_t)Geo::mat_bytes;
  bf16* sW = smem; bf16* sX = smem + 2 * UIMG; bf16* sP = smem + 4 * UIMG;
  const int tid = threadIdx.x;
  const int row = Geo::row(), col0 = Geo::col0();
  const bool act = Geo::active();
  umma_begin(ctl, UM);
  uint32_t phase = 0;
  // W + eps I staged in fp32 in the space of Q: norms, images of W and X_0, fp32 X_0 all come from there
  float* Wf = reinterpret_cast<float*>(sP);      // [UM][UM], pitch UM
#pragma unroll 1
  for (int b0 = 0; b0 < UM * UM / 256; b0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = (b0 + u) * 256 + tid, i = e >> LOG, j = e & (UM - 1);
      v[u] = (i < m && j < m) ? W[(long long)i * m + j] + (i == j ? eps : 0.f) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) Wf[(b0 + u) * 256 + tid] = v[u];
  }
  __syncthreads();
  {
    float* colsum = red; float* rowsum = red + 256;
    if (tid < m) {
      float cs = 0.f, rs = 0.f;
      for (int i = 0; i < m; ++i) cs += fabsf(Wf[i * UM + tid]);
      for (int i = 0; i < UM; ++i) rs += fabsf(Wf[tid * UM + ((i + tid) & (UM - 1))]);   // rotated start: no bank conflicts; padding is zero
      colsum[tid] = cs; rowsum[tid] = rs;
    }
    __syncthreads();
    if (tid == 0) {
      float n1, ninf; int js, is;
      norm_argmax(colsum, m, n1, js);
      norm_argmax(rowsum, m, ninf, is);
      hdr->n1 = n1; hdr->ninf = ninf; hdr->jstar = js; hdr->istar = is;
      hdr->auto_alpha = !(alpha_in > 0.f);
      hdr->alpha = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * ninf);
      hdr->pad0 = hdr->pad1 = 0;
    }
    __syncthreads();
  }
  const float alpha = hdr->alpha;
  if (act) {  // this thread's row: NV columns of W and of X_0 = alpha W^T
    float w[NV], x0[NV];
#pragma unroll
    for (int q = 0; q < NV; ++q) { w[q] = Wf[row * UM + col0 + q]; x0[q] = alpha * Wf[(col0 + q) * UM + row]; }
    umma_row_to_image<UM>(w, row, col0, sW);
    umma_row_to_image<UM>(x0, row, col0, sX);
    if (T == 0 && row < m) umma_row_to_global<NV>(x0, Xh + (long long)row * ld, col0, ld);
    if (T == 0) {
#pragma unroll
      for (int q = 0; q < NV; ++q) bad += isfinite(x0[q]) ? 0.f : 1.f;
    }
  }
  bool ok = true;
  umma_step_done(ctl, true);
  if (tid == 0 && T > 0) umma::bulk_store(Xh, sX, MATB);                                   // image of X_0
  for (int k = 0; k < T; ++k) {
    // the store of Q_{k-1} has read sP before the barrier of this product completes
    ok &= umma_run<UM>(ctl, phase, ctl.tmem_base, sW, true, sX, false, false, nullptr, true, nullptr, true, true);   // D = W X_k
    {
      float v[NV];
      umma_row<NV>(ctl.tmem_base, col0, v);
      if (act) {
#pragma unroll
        for (int q = 0; q < NV; ++q) v[q] = ((row == col0 + q && row < m) ? 2.f : 0.f) - v[q];   // Q_k = 2I - W X_k
        umma_row_to_image<UM>(v, row, col0, sP);
      }
    }
    umma_step_done(ctl, ok);
    if (tid == 0 && Ph) umma::bulk_store(Ph + k * hs, sP, MATB);
    // the store of X_k has read sX before the barrier of this product completes
    ok &= umma_run<UM>(ctl, phase, ctl.tmem_base, sX, true, sP, false, false, nullptr, true, nullptr, true, true);   // D = X_k Q_k
    {
      float v[NV];
      umma_row<NV>(ctl.tmem_base, col0, v);
      if (act) {
        if (k + 1 == T) {
          if (row < m) umma_row_to_global<NV>(v, Xh + T * hs + (long long)row * ld, col0, ld);
#pragma unroll
          for (int q = 0; q < NV; ++q) bad += isfinite(v[q]) ? 0.f : 1.f;
        }
        umma_row_to_image<UM>(v, row, col0, sX);     // the MMAs and the bulk store that read X_k have completed
      }
    }
    umma_step_done(ctl, ok);
    if (tid == 0 && k + 1 < T) umma::bulk_store(Xh + (k + 1) * hs, sX, MATB);
  }
  if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // every image has reached global memory
  ok &= (ctl.timeout == 0);
  umma_end(ctl, UM);
  return ok;
}

// Adjoint of the iteration for a symmetric W (the landmark kernel matrix is symmetric bit for bit).
// Per step k (A = X_k, Q = 2I - W A, both saved as operand images by the forward pass):
//     H = A^T G,   dW -= H A^T,   G <- G Q^T + Q^T G - 2G.
// In general the last term of the step adjoint is W^T H = (A W)^T G; for symmetric W every iterate is a
// polynomial in W, so A W = W A up to rounding, (A W)^T G = (2I - Q)^T G, and W itself is not needed inside
// the loop.  G is kept in fp32 in registers and re-split into its image after each update.
// smem: images A (also used for Q), G, H.  TMEM: UM columns for the running product, UM for dW accumulated over
// all steps.  The images arrive by bulk copies on an mbarrier; the copy of the next A runs beside the G update.
// UM = 64 has room for a fourth image: Q has its own buffer, A and Q of the next step are both fetched ahead, and
// the products dW += H A^T and G Q^T + Q^T G are issued together and waited for once (two waits per step, not three).
// Output: GW [m][ldgw] = (dW o W + (dW o W)^T) / lambda, the upstream of the landmark kernel block (dW itself
// stays on chip).
template <int UM>
__device__ bool ns_backward_umma(int m, int T, float eps, const float* W, const float* Xh, const float* Ph, int ld,
                                 long long hs, const NsHdr* hdr, const float* G0, float* GW, int ldgw, float inv_lambda,
                                 bf16* smem, float* red, UmmaCtl& ctl) {
  typedef UmmaGeo<UM> Geo;
  constexpr int UIMG = Geo::UIMG, NV = Geo::NV, LOG = Geo::LOG;
  constexpr uint32_t MATB = (uint32_t)Geo::mat_bytes;
  constexpr bool QBUF = (UM == 64);
  bf16* sA = smem; bf16* sG = smem + 2 * UIMG; bf16* sH = smem + 4 * UIMG; bf16* sQ = smem + (QBUF ? 6 : 0) * UIMG;
  const int tid = threadIdx.x;
  const int row = Geo::row(), col0 = Geo::col0();
  const bool act = Geo::active();
  umma_begin(ctl, 2 * UM);
  uint32_t phase = 0, ph_ld = 0;
  const uint32_t t_acc = ctl.tmem_base, t_dw = ctl.tmem_base + UM;
  auto load_image = [&](const float* src) {     // one thread starts the copy into sA
    if (tid == 0) {
      umma::mbar_expect_tx(&ctl.mbar_ld, MATB);
      umma::bulk_load(sA, src, MATB, &ctl.mbar_ld);
    }
  };
  auto wait_image = [&]() {                     // everybody sees the image (thread 0 issues the MMAs that read it)
    const bool got = umma::mbar_wait(&ctl.mbar_ld, ph_ld & 1);
    ph_ld ^= 1u;
    return got;
  };
  auto load_pair = [&](int k) {                 // A = X_k and Q_k, counted on one phase of the barrier
    if (tid == 0) {
      umma::mbar_expect_tx(&ctl.mbar_ld, 2 * MATB);
      umma::bulk_load(sA, Xh + (long long)k * hs, MATB, &ctl.mbar_ld);
      umma::bulk_load(sQ, Ph + (long long)k * hs, MATB, &ctl.mbar_ld);
    }
  };
  if (T > 0) { if constexpr (QBUF) load_pair(T - 1); else load_image(Xh + (long long)(T - 1) * hs); }
  float G[NV];                                 // this thread's part of G in full precision
#pragma unroll
  for (int q = 0; q < NV; ++q) G[q] = (act && row < m && col0 + q < m) ? G0[(long long)row * ld + col0 + q] : 0.f;
  if (act) umma_row_to_image<UM>(G, row, col0, sG);
  bool ok = true;
  for (int k = T - 1; k >= 0; --k) {
    ok &= wait_image();                                                                       // A = X_k
    umma_step_done(ctl, ok);
    ok &= umma_run<UM>(ctl, phase, t_acc, sA, false, sG, false, false);                      // H = A^T G
    {
      float v[NV];
      umma_row<NV>(t_acc, col0, v);
      if (act) umma_row_to_image<UM>(v, row, col0, sH);
    }
    umma_step_done(ctl, ok);
    if constexpr (QBUF) {
      if (tid == 0) {
        umma::fence_after_sync();
        umma_gemm<UM>(t_dw, sH, true, sA, true, k != T - 1);                                  // dW accumulator += H A^T
        umma_gemm<UM>(t_acc, sG, true, sQ, true, false);                                      // G Q^T
        umma_gemm<UM>(t_acc, sQ, false, sG, false, true);                                     //   + Q^T G
        umma::commit(&ctl.mbar);
      }
      ok &= umma::mbar_wait(&ctl.mbar, phase & 1);
      phase ^= 1u;
      umma::fence_after_sync();
      if (k > 0) load_pair(k - 1);                                                            // next A and Q, beside the G update
    } else {
      ok &= umma_run<UM>(ctl, phase, t_dw, sH, true, sA, true, k != T - 1);                  // dW accumulator += H A^T
      load_image(Ph + (long long)k * hs);                                                     // Q_k (A is no longer read)
      ok &= wait_image();
      umma_step_done(ctl, ok);
      ok &= umma_run<UM>(ctl, phase, t_acc, sG, true, sA, true, false, sA, false, sG, false);   // G Q^T + Q^T G
      if (k > 0) load_image(Xh + (long long)(k - 1) * hs);                                    // next A, beside the G update
    }
    {
      float v[NV];
      umma_row<NV>(t_acc, col0, v);
      if (act) {
#pragma unroll
        for (int q = 0; q < NV; ++q) G[q] = (row < m && col0 + q < m) ? v[q] - 2.f * G[q] : 0.f;
        umma_row_to_image<UM>(G, row, col0, sG);
      }
    }
  }
  umma_step_done(ctl, ok);
  float dw[NV];                                // this thread's part of -(accumulated H A^T)
  {
    float v[NV];
    if (T > 0) umma_row<NV>(t_dw, col0, v);
#pragma unroll
    for (int q = 0; q < NV; ++q) dw[q] = (T > 0) ? -v[q] : 0.f;
  }
  ok &= (ctl.timeout == 0);
  umma_end(ctl, 2 * UM);
  __syncthreads();
  // End of the adjoint and the upstream of the landmark block, from shared memory (the operand buffers are free):
  //   X_0 = alpha (W + eps I)^T:  d alpha = <G, Wr^T>,  dW += alpha G^T, then the alpha(W) terms;
  //   GW = (dW o W + (dW o W)^T) / lambda.
  // G and Wr are staged as fp32 [UM][UM + 1] (the odd pitch makes the transposed reads conflict-free).
  constexpr int PT = UM + 1;
  float* sGf = reinterpret_cast<float*>(smem);
  float* sWf = sGf + UM * PT;
  if (act) {
#pragma unroll
    for (int q = 0; q < NV; ++q) sGf[row * PT + col0 + q] = G[q];
  }
  for (int e = tid; e < UM * UM; e += 256) {
    const int i = e >> LOG, j = e & (UM - 1);
    sWf[i * PT + j] = (i < m && j < m) ? W[(long long)i * m + j] + (i == j ? eps : 0.f) : 0.f;
  }
  __syncthreads();
  const float alpha = hdr->alpha;
  float part = 0.f;
  if (act) {
#pragma unroll
    for (int q = 0; q < NV; ++q) part += G[q] * sWf[(col0 + q) * PT + row];
  }
  const float dalpha = block_sum(part, red);
  const bool aa = hdr->auto_alpha != 0;
  const int js = hdr->jstar, is = hdr->istar;
  const float c1 = dalpha * (-alpha / hdr->n1), c2 = dalpha * (-alpha / hdr->ninf);
  if (act) {
#pragma unroll
    for (int q = 0; q < NV; ++q) {
      const int j = col0 + q;
      float v = dw[q] + alpha * sGf[j * PT + row];
      if (aa) {
        const float w = sWf[row * PT + j];
        const float sg = w > 0.f ? 1.f : (w < 0.f ? -1.f : 0.f);
        if (j == js) v += c1 * sg;
        if (row == is) v += c2 * sg;
      }
      dw[q] = (row < m && j < m) ? v : 0.f;
    }
  }
  __syncthreads();                             // everybody has read G
  if (act) {
#pragma unroll
    for (int q = 0; q < NV; ++q) sGf[row * PT + col0 + q] = dw[q];      // now dW
  }
  __syncthreads();
  if (act && row < m) {
    float* grow = GW + (long long)row * ldgw;
#pragma unroll
    for (int q = 0; q < NV; q += 4) {
      const int j = col0 + q;
      if (j >= ldgw) break;
      float o[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int jj = j + u;
        o[u] = (jj < m) ? (dw[q + u] * sWf[row * PT + jj] + sGf[jj * PT + row] * sWf[jj * PT + row]) * inv_lambda : 0.f;
      }
      *reinterpret_cast<float4*>(grow + j) = make_float4(o[0], o[1], o[2], o[3]);
    }
  }
  return ok;
}

}  // namespace ln
