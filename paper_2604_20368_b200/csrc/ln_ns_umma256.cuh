// Newton-Schulz (Alg. 2) and its adjoint for 128 < m <= 256 on the 5th-generation tensor cores.
//
// The matrix is padded with zeros to 256 x 256 and cut into 2 x 2 blocks of 128 x 128.  Four CTAs of a
// thread-block cluster share a head; CTA c owns the output block (ri, ci) = (c / 2, c % 2) of every product:
//     D[ri][ci] = sum_kb  A[ri][kb] B[kb][ci]          (two block products into one TMEM accumulator)
// Every matrix of the iteration lives in global memory (L2) as four operand images (bf16 hi + lo in the
// canonical core-matrix layout, 64 KiB per block, 256 KiB per matrix): a CTA fetches the two blocks of a term
// with bulk copies on an mbarrier, issues tcgen05.mma (three MMAs per term: lo*hi, hi*lo, hi*hi), reads its
// accumulator with tcgen05.ld, writes the image of its output block to shared memory and sends it to global
// memory with a bulk copy; the cluster barrier ends a phase, after which every CTA may fetch what the others
// wrote.  The images the forward pass leaves (X_k, Q_k = 2I - W X_k) are the history the adjoint fetches.
// Transposes cost nothing: an image is read K-major or MN-major through the descriptor.
//
// Shared memory: three 64 KiB buffers, operand blocks in rotation and the output image (sC).  Thread t owns row
// 32 (warp % 4) + lane of its CTA's block and the column half warp / 4 (as on the 128 x 128 path).
// Every wait is bounded; a wait that runs out is reported to the caller (results are then wrong, nothing hangs:
// all threads of all four CTAs still reach every cluster barrier).
#pragma once
#include "ln_ns_umma.cuh"

namespace ln {

constexpr int U2 = 256;                                   // padded matrix size of this path
constexpr long long kU2Slot = (long long)U2 * U2;         // floats per matrix slot: four block images, or fp32 [m][m]
constexpr int kU2BlockFloats = (int)(kUmmaMatBytes / 4);  // floats per block image

// block (bi, bj) of the images in a slot
__device__ __forceinline__ const bf16* u2_block(const float* slot, int bi, int bj) {
  return reinterpret_cast<const bf16*>(slot + (long long)(bi * 2 + bj) * kU2BlockFloats);
}
__device__ __forceinline__ float* u2_block_w(float* slot, int bi, int bj) { return slot + (long long)(bi * 2 + bj) * kU2BlockFloats; }

// one term of a product: A block, B block (global images), how each is read, where it accumulates
struct U2Term { const bf16* A; bool a_k; const bf16* B; bool b_k; uint32_t tmem_d; bool accumulate; };

struct U2Ctx {
  UmmaCtl* ctl; unsigned long long* mbar_free;   // mbar_free: the MMAs that read sA / sB have completed
  bf16 *sA, *sB, *sC;
  uint32_t phase, ph_ld, ph_free;               // ph_ld / ph_free are used by thread 0 only
  bool ok;
};

// Writes of other CTAs to global memory (bulk copies, then the cluster barrier) are read here by bulk copies.
__device__ __forceinline__ void u2_fence_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// All terms, one after the other; one thread fetches and issues, everybody waits for the last MMA.  The three buffers
// (all free between products: the output image is written after the last MMA) rotate so that the A block of the next
// term is fetched while the MMAs of this one run; its B block follows as soon as they have completed.
//   term i: A in buffer 2i mod 3, B in buffer (2i + 1) mod 3
template <int NT>
__device__ __forceinline__ void u2_run(U2Ctx& c, const U2Term (&t)[NT]) {
  constexpr uint32_t MATB = (uint32_t)kUmmaMatBytes;
  if (threadIdx.x == 0) {
    bf16* const buf[3] = {c.sA, c.sB, c.sC};
    u2_fence_async();
    umma::mbar_expect_tx(&c.ctl->mbar_ld, 2 * MATB);
    umma::bulk_load(buf[0], t[0].A, MATB, &c.ctl->mbar_ld);
    umma::bulk_load(buf[1], t[0].B, MATB, &c.ctl->mbar_ld);
#pragma unroll 1
    for (int i = 0; i < NT; ++i) {
      const int ia = (2 * i) % 3, ib = (2 * i + 1) % 3;
      c.ok &= umma::mbar_wait(&c.ctl->mbar_ld, c.ph_ld & 1);
      c.ph_ld ^= 1u;
      umma::fence_after_sync();
      umma_gemm<128>(t[i].tmem_d, buf[ia], t[i].a_k, buf[ib], t[i].b_k, t[i].accumulate);
      if (i + 1 < NT) {
        umma::mbar_expect_tx(&c.ctl->mbar_ld, 2 * MATB);
        umma::bulk_load(buf[(2 * i + 2) % 3], t[i + 1].A, MATB, &c.ctl->mbar_ld);   // free since term i - 1 completed
        umma::commit(c.mbar_free);                                                   // term i has finished reading
        c.ok &= umma::mbar_wait(c.mbar_free, c.ph_free & 1);
        c.ph_free ^= 1u;
        umma::bulk_load(buf[(2 * i + 3) % 3], t[i + 1].B, MATB, &c.ctl->mbar_ld);   // the buffer of this term's A
      }
    }
    umma::commit(&c.ctl->mbar);
    if (!c.ok) c.ctl->timeout = 1;
  }
  c.ok &= umma::mbar_wait(&c.ctl->mbar, c.phase & 1);
  c.phase ^= 1u;
  umma::fence_after_sync();
}

// This thread's 64 values -> image in sC; then one thread sends the image to `dst` (a block in global memory) and waits
// until it has arrived.  Ends with a CTA barrier (sC may be rewritten, the accumulator may be overwritten).
__device__ __forceinline__ void u2_store_block(U2Ctx& c, const float (&v)[64], int row, int col0, float* dst) {
  umma_row_to_image<128>(v, row, col0, c.sC);
  umma::fence_smem_to_mma();
  umma::fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0) {
    umma::bulk_store(dst, c.sC, (uint32_t)kUmmaMatBytes);
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    u2_fence_async();
  }
  __syncthreads();
}

__device__ __forceinline__ void u2_begin(U2Ctx& c, UmmaCtl& ctl, unsigned long long* mbar_free, bf16* smem, int ncols) {
  c.ctl = &ctl; c.mbar_free = mbar_free;
  c.sA = smem; c.sB = smem + 2 * UmmaGeo<128>::UIMG; c.sC = smem + 4 * UmmaGeo<128>::UIMG;
  c.phase = c.ph_ld = c.ph_free = 0; c.ok = true;
  if (threadIdx.x == 0) umma::mbar_init(mbar_free, 1);
  umma_begin(ctl, ncols);
}

// Forward iteration, called by the four CTAs of a cluster (crank = 0 .. 3).  W: fp32 [m][m]; Wr: unused (W + eps I is
// formed where it is read); Wimg: scratch slot for the images of Wr; Xh: slots 0 .. T-1 receive the images of X_k, slot T
// X_T in fp32 [m][m]; Ph: slot k receives the images of Q_k.  Returns false if a wait ran out.
__device__ bool ns_forward_umma256(int m, int T, float eps, float alpha_in, const float* W, float* Wr, float* Wimg,
                                   float* Xh, float* Ph, NsHdr* hdr, bf16* smem, float* red, UmmaCtl& ctl,
                                   unsigned long long* mbar_free, int crank, float& bad) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int ri = crank >> 1, ci = crank & 1;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64;
  const int gi = ri * 128 + row, gj0 = ci * 128 + col0;          // this thread's row and first column in the matrix
  // Wr = W + eps I is never written out on this path: the ridge is added where an element of the diagonal is read
  (void)Wr;
  {
    // Norms: Wr is symmetric bit for bit (|a - b| = |b - a| term by term in the kernel block), so the absolute row sums
    // are the absolute column sums; a column is read along the rows (threads side by side), sixteen rows in flight.
    float* colsum = red;
    if (tid < m) {
      float c16[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) c16[u] = 0.f;
      int i = 0;
      for (; i + 15 < m; i += 16) {
        float w16[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) w16[u] = W[(long long)(i + u) * m + tid];
#pragma unroll
        for (int u = 0; u < 16; ++u) c16[u] += fabsf(w16[u] + (i + u == tid ? eps : 0.f));
      }
      for (; i < m; ++i) c16[0] += fabsf(W[(long long)i * m + tid] + (i == tid ? eps : 0.f));
#pragma unroll
      for (int o = 8; o > 0; o >>= 1)
#pragma unroll
        for (int u = 0; u < o; ++u) c16[u] += c16[u + o];
      colsum[tid] = c16[0];
    }
    __syncthreads();
    if (tid == 0) {               // every CTA of the cluster arrives at the same values
      float n1; int js;
      norm_argmax(colsum, m, n1, js);                            // near-ties (duplicated landmarks): the lowest index
      red[512] = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * n1);
      if (crank == 0) {
        hdr->n1 = n1; hdr->ninf = n1; hdr->jstar = js; hdr->istar = js;
        hdr->auto_alpha = !(alpha_in > 0.f);
        hdr->alpha = red[512];
        hdr->pad0 = hdr->pad1 = 0;
      }
    }
    __syncthreads();
  }
  const float alpha = red[512];
  U2Ctx c;
  u2_begin(c, ctl, mbar_free, smem, 128);
  const uint32_t t_acc = ctl.tmem_base;
  {  // images of this CTA's block of Wr and of X_0 = alpha Wr^T
    float v[64];
#pragma unroll
    for (int q = 0; q < 64; ++q) v[q] = (gi < m && gj0 + q < m) ? W[(long long)gi * m + gj0 + q] + (gi == gj0 + q ? eps : 0.f) : 0.f;
    u2_store_block(c, v, row, col0, u2_block_w(Wimg, ri, ci));
#pragma unroll
    for (int q = 0; q < 64; ++q) v[q] = (gi < m && gj0 + q < m) ? alpha * (W[(long long)(gj0 + q) * m + gi] + (gi == gj0 + q ? eps : 0.f)) : 0.f;
    if (T == 0) {
      if (gi < m) {
#pragma unroll
        for (int q = 0; q < 64; ++q) if (gj0 + q < m) Xh[(long long)gi * m + gj0 + q] = v[q];
      }
#pragma unroll
      for (int q = 0; q < 64; ++q) bad += isfinite(v[q]) ? 0.f : 1.f;
    } else {
      u2_store_block(c, v, row, col0, u2_block_w(Xh, ri, ci));
    }
  }
  phase_sync<4>();
  for (int k = 0; k < T; ++k) {
    const float* X = Xh + (long long)k * kU2Slot;
    float* Q = Ph + (long long)k * kU2Slot;
    {  // Q_k = 2I - Wr X_k
      const U2Term t[2] = {{u2_block(Wimg, ri, 0), true, u2_block(X, 0, ci), false, t_acc, false},
                           {u2_block(Wimg, ri, 1), true, u2_block(X, 1, ci), false, t_acc, true}};
      u2_run<2>(c, t);
      float v[64];
      umma_row<64>(t_acc, col0, v);
#pragma unroll
      for (int q = 0; q < 64; ++q) v[q] = ((gi == gj0 + q && gi < m) ? 2.f : 0.f) - v[q];
      u2_store_block(c, v, row, col0, u2_block_w(Q, ri, ci));
    }
    phase_sync<4>();
    {  // X_{k+1} = X_k Q_k
      const U2Term t[2] = {{u2_block(X, ri, 0), true, u2_block(Q, 0, ci), false, t_acc, false},
                           {u2_block(X, ri, 1), true, u2_block(Q, 1, ci), false, t_acc, true}};
      u2_run<2>(c, t);
      float v[64];
      umma_row<64>(t_acc, col0, v);
      float* Xn = Xh + (long long)(k + 1) * kU2Slot;
      if (k + 1 == T) {
        if (gi < m) {
#pragma unroll
          for (int q = 0; q < 64; q += 4)
            if (gj0 + q < m) {       // m is a multiple of 4 on this path's callers only by chance: element-wise tail
              if (gj0 + q + 3 < m && (m & 3) == 0) *reinterpret_cast<float4*>(Xn + (long long)gi * m + gj0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
              else for (int u = 0; u < 4; ++u) if (gj0 + q + u < m) Xn[(long long)gi * m + gj0 + q + u] = v[q + u];
            }
        }
#pragma unroll
        for (int q = 0; q < 64; ++q) bad += isfinite(v[q]) ? 0.f : 1.f;
        umma::fence_before_sync();
        __syncthreads();
      } else {
        u2_store_block(c, v, row, col0, u2_block_w(Xn, ri, ci));
      }
    }
    phase_sync<4>();
  }
  const bool ok = c.ok && ctl.timeout == 0;
  umma_end(ctl, 128);
  return ok;
}

// Adjoint for a symmetric W (same algebra as the 128 x 128 path): per step k, with A = X_k and Q = Q_k as the forward
// pass left them,  H = A^T G,  dW -= H A^T,  G <- G Q^T + Q^T G - 2G.  G0 = dLoss/dX_T, fp32 [m][m].  Scratch slots
// (kU2Slot floats each): Gimg0, Gimg1 (images of G, alternating), Himg.  Outputs, fp32 [m][m]: Gout = dLoss/dX_0 and
// dW = -(sum over the steps of H A^T).  Returns false if a wait ran out.
__device__ bool ns_backward_umma256(int m, int T, const float* Xh, const float* Ph, const float* G0, float* Gimg0,
                                    float* Gimg1, float* Himg, float* Gout, float* dW, bf16* smem, UmmaCtl& ctl,
                                    unsigned long long* mbar_free, int crank) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int ri = crank >> 1, ci = crank & 1;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64;
  const int gi = ri * 128 + row, gj0 = ci * 128 + col0;
  U2Ctx c;
  u2_begin(c, ctl, mbar_free, smem, 256);
  const uint32_t t_acc = ctl.tmem_base, t_dw = ctl.tmem_base + 128;
  float G[64];
#pragma unroll
  for (int q = 0; q < 64; ++q) G[q] = (gi < m && gj0 + q < m) ? G0[(long long)gi * m + gj0 + q] : 0.f;
  float* Gcur = Gimg0; float* Gnext = Gimg1;
  if (T > 0) u2_store_block(c, G, row, col0, u2_block_w(Gcur, ri, ci));
  phase_sync<4>();
  for (int k = T - 1; k >= 0; --k) {
    const float* A = Xh + (long long)k * kU2Slot;
    const float* Q = Ph + (long long)k * kU2Slot;
    {  // H = A^T G:  H[ri][ci] = sum_kb (A[kb][ri])^T G[kb][ci]
      const U2Term t[2] = {{u2_block(A, 0, ri), false, u2_block(Gcur, 0, ci), false, t_acc, false},
                           {u2_block(A, 1, ri), false, u2_block(Gcur, 1, ci), false, t_acc, true}};
      u2_run<2>(c, t);
      float v[64];
      umma_row<64>(t_acc, col0, v);
      u2_store_block(c, v, row, col0, u2_block_w(Himg, ri, ci));
    }
    phase_sync<4>();
    {  // dW accumulator += H A^T;  G Q^T + Q^T G
      const bool acc = k != T - 1;
      const U2Term t[6] = {{u2_block(Himg, ri, 0), true, u2_block(A, ci, 0), true, t_dw, acc},
                           {u2_block(Himg, ri, 1), true, u2_block(A, ci, 1), true, t_dw, true},
                           {u2_block(Gcur, ri, 0), true, u2_block(Q, ci, 0), true, t_acc, false},
                           {u2_block(Gcur, ri, 1), true, u2_block(Q, ci, 1), true, t_acc, true},
                           {u2_block(Q, 0, ri), false, u2_block(Gcur, 0, ci), false, t_acc, true},
                           {u2_block(Q, 1, ri), false, u2_block(Gcur, 1, ci), false, t_acc, true}};
      u2_run<6>(c, t);
      float v[64];
      umma_row<64>(t_acc, col0, v);
#pragma unroll
      for (int q = 0; q < 64; ++q) G[q] = (gi < m && gj0 + q < m) ? v[q] - 2.f * G[q] : 0.f;
      if (k > 0) u2_store_block(c, G, row, col0, u2_block_w(Gnext, ri, ci));
      else { umma::fence_before_sync(); __syncthreads(); }
    }
    phase_sync<4>();
    float* tsw = Gcur; Gcur = Gnext; Gnext = tsw;
  }
  {
    float v[64];
    if (T > 0) umma_row<64>(t_dw, col0, v);
    if (gi < m) {
#pragma unroll
      for (int q = 0; q < 64; ++q)
        if (gj0 + q < m) {
          Gout[(long long)gi * m + gj0 + q] = G[q];
          dW[(long long)gi * m + gj0 + q] = (T > 0) ? -v[q] : 0.f;
        }
    }
  }
  const bool ok = c.ok && ctl.timeout == 0;
  umma_end(ctl, 256);
  phase_sync<4>();
  return ok;
}

}  // namespace ln
