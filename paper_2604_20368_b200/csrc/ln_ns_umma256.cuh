// Newton-Schulz (Alg. 2) and its adjoint for 128 < m <= 256 on the 5th-generation tensor cores.
//
// The matrix is padded with zeros to 256 x 256 and cut into 2 x 2 blocks of 128 x 128.  Two CTAs of a
// thread-block cluster share a head; CTA ri owns the block row ri of every product, both column blocks:
//     D[ri][ci] = sum_kb  A[ri][kb] B[kb][ci],   ci = 0, 1      (two TMEM accumulators of 128 columns)
// Every matrix of the iteration lives in global memory (L2) as four operand images (bf16 hi + lo in the
// canonical core-matrix layout, 64 KiB per block, 256 KiB per matrix).  The work of a product is a list of
// GROUPS: one block S on the A side and the two blocks x, y it multiplies, S x -> accumulator 0, S y ->
// accumulator 1 (three MMAs per block product: lo*hi, hi*lo, hi*hi).  A CTA fetches the three blocks of a group
// with bulk copies on an mbarrier into its three 64 KiB buffers; as soon as S x has completed, the S block of the
// next group is fetched into x's buffer, and as soon as S y has completed, the next x and y go into the other
// two, S x of that group starting as soon as its S and x are there, while y still arrives: every A-side block is
// fetched once for both column blocks, and two of three fetches run beside MMAs.
// After the last group the threads read both accumulators with tcgen05.ld, write the images of the two output
// blocks to shared memory and send them to global memory with bulk copies; the cluster barrier ends a phase,
// after which every CTA may fetch what the other wrote.  The images the forward pass leaves (X_k,
// Q_k = 2I - W X_k) are the history the adjoint fetches.  Transposes cost nothing: an image is read K-major or
// MN-major through the descriptor.
//
// Thread t owns row 32 (warp % 4) + lane of a block and the column half warp / 4 (as on the 128 x 128 path).
// Every wait is bounded; a wait that runs out is reported to the caller (results are then wrong, nothing hangs:
// all threads of both CTAs still reach every cluster barrier).
#pragma once
#include "ln_ns_umma.cuh"

namespace ln {

constexpr int U2 = 256;                                   // padded matrix size of this path
constexpr int kU2Cluster = 2;                             // CTAs that share a head
constexpr long long kU2Slot = (long long)U2 * U2;         // floats per matrix slot: four block images, or fp32 [m][m]
constexpr int kU2BlockFloats = (int)(kUmmaMatBytes / 4);  // floats per block image

// block (bi, bj) of the images in a slot
__device__ __forceinline__ const bf16* u2_block(const float* slot, int bi, int bj) {
  return reinterpret_cast<const bf16*>(slot + (long long)(bi * 2 + bj) * kU2BlockFloats);
}
__device__ __forceinline__ float* u2_block_w(float* slot, int bi, int bj) { return slot + (long long)(bi * 2 + bj) * kU2BlockFloats; }

// one group of a product: the A-side block S (how it is read), the two B-side blocks it multiplies (how they are
// read; Y may be NULL: one block product only), the two accumulators, and whether they are added to
struct U2Group { const bf16* S; bool s_k; const bf16* X; const bf16* Y; bool b_k; uint32_t d0, d1; bool accumulate; };

struct U2Ctx {
  UmmaCtl* ctl; unsigned long long* mbar_x; unsigned long long* mbar_y;   // S x has completed; S y (and S x) have completed
  unsigned long long* mbar_ldy;                 // arrival of the y block (S and x are counted on ctl->mbar_ld)
  bf16* buf[3];
  uint32_t phase, ph_ld, ph_ldy, ph_x, ph_y;    // ph_ld / ph_ldy / ph_x / ph_y are used by thread 0 only
  bool pre;                                     // thread 0: the first S block of the next product is on its way into buffer 2
  bool ok;
};

// Writes of other CTAs to global memory (bulk copies, then the cluster barrier) are read here by bulk copies.
__device__ __forceinline__ void u2_fence_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// All groups, one after the other; one thread fetches and issues, everybody waits for the last MMA.  Buffers 0 and 1
// are free on entry (the output images of the previous product have left); buffer 2 is free, or already receives the
// first S block (see next_S).
// next_S: NULL, or the first S block of the NEXT call, which must not depend on what this product or the other CTA is
// still writing: its fetch into buffer 2 starts as soon as the last MMA of this call has completed and runs beside the
// epilogue (which stages the output images in buffers 0 and 1) and the cluster barrier.
template <int NG>
__device__ __forceinline__ void u2_run(U2Ctx& c, const U2Group (&g)[NG], const bf16* next_S = nullptr) {
  constexpr uint32_t MATB = (uint32_t)kUmmaMatBytes;
  if (threadIdx.x == 0) {
    int is = 0, ix = 1, iy = 2;                                       // buffers of S, x, y of the current group
    u2_fence_async();
    if (c.pre) {                                                       // S is on its way (its bytes and x's were announced then)
      is = 2; ix = 0; iy = 1;
    } else {
      umma::mbar_expect_tx(&c.ctl->mbar_ld, 2 * MATB);
      umma::bulk_load(c.buf[is], g[0].S, MATB, &c.ctl->mbar_ld);
    }
    umma::bulk_load(c.buf[ix], g[0].X, MATB, &c.ctl->mbar_ld);
    if (g[0].Y) {
      umma::mbar_expect_tx(c.mbar_ldy, MATB);
      umma::bulk_load(c.buf[iy], g[0].Y, MATB, c.mbar_ldy);
    }
#pragma unroll 1
    for (int i = 0; i < NG; ++i) {
      c.ok &= umma::mbar_wait(&c.ctl->mbar_ld, c.ph_ld & 1);         // S and x are here: S x starts while y is still arriving
      c.ph_ld ^= 1u;
      umma::fence_after_sync();
      umma_gemm<128>(g[i].d0, c.buf[is], g[i].s_k, c.buf[ix], g[i].b_k, g[i].accumulate);
      if (i + 1 < NG) umma::commit(c.mbar_x);
      if (g[i].Y) {                                                    // a group may have one B-side block only
        c.ok &= umma::mbar_wait(c.mbar_ldy, c.ph_ldy & 1);
        c.ph_ldy ^= 1u;
        umma::fence_after_sync();
        umma_gemm<128>(g[i].d1, c.buf[is], g[i].s_k, c.buf[iy], g[i].b_k, g[i].accumulate);
      }
      if (i + 1 < NG) {
        umma::commit(c.mbar_y);
        c.ok &= umma::mbar_wait(c.mbar_x, c.ph_x & 1);               // x's buffer has been read
        c.ph_x ^= 1u;
        umma::mbar_expect_tx(&c.ctl->mbar_ld, 2 * MATB);               // S and x of the next group, counted together
        umma::bulk_load(c.buf[ix], g[i + 1].S, MATB, &c.ctl->mbar_ld);
        c.ok &= umma::mbar_wait(c.mbar_y, c.ph_y & 1);               // S's and y's buffers have been read
        c.ph_y ^= 1u;
        umma::bulk_load(c.buf[is], g[i + 1].X, MATB, &c.ctl->mbar_ld);
        if (g[i + 1].Y) {
          umma::mbar_expect_tx(c.mbar_ldy, MATB);
          umma::bulk_load(c.buf[iy], g[i + 1].Y, MATB, c.mbar_ldy);
        }
        const int t = is; is = ix; ix = t;                             // the next S sits where x was, the next x where S was
      }
    }
    umma::commit(&c.ctl->mbar);
    if (!c.ok) c.ctl->timeout = 1;
  }
  c.ok &= umma::mbar_wait(&c.ctl->mbar, c.phase & 1);
  c.phase ^= 1u;
  umma::fence_after_sync();
  if (threadIdx.x == 0) {
    c.pre = next_S != nullptr;
    if (next_S) {                                                      // every buffer has been read; the epilogue uses 0 and 1
      umma::mbar_expect_tx(&c.ctl->mbar_ld, 2 * MATB);
      umma::bulk_load(c.buf[2], next_S, MATB, &c.ctl->mbar_ld);
    }
  }
}

// This thread's 64 values of a block -> image in buffer `b`; then one thread sends the image to `dst` (a block in
// global memory).  With `last` the thread also waits until every image it sent has arrived and fences, and the call
// ends with a CTA barrier (the buffers may be rewritten, the accumulators overwritten).
__device__ __forceinline__ void u2_store_block(U2Ctx& c, const float (&v)[64], int row, int col0, float* dst, int b, bool last) {
  umma_row_to_image<128>(v, row, col0, c.buf[b]);
  umma::fence_smem_to_mma();
  umma::fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0) {
    umma::bulk_store(dst, c.buf[b], (uint32_t)kUmmaMatBytes);
    if (last) {
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      u2_fence_async();
    }
  }
  if (last) __syncthreads();
}

__device__ __forceinline__ void u2_begin(U2Ctx& c, UmmaCtl& ctl, unsigned long long* mbars, bf16* smem, int ncols) {
  c.ctl = &ctl; c.mbar_x = mbars; c.mbar_y = mbars + 1; c.mbar_ldy = mbars + 2;
  c.buf[0] = smem; c.buf[1] = smem + 2 * UmmaGeo<128>::UIMG; c.buf[2] = smem + 4 * UmmaGeo<128>::UIMG;
  c.phase = c.ph_ld = c.ph_ldy = c.ph_x = c.ph_y = 0; c.ok = true; c.pre = false;
  if (threadIdx.x == 0) { umma::mbar_init(mbars, 1); umma::mbar_init(mbars + 1, 1); umma::mbar_init(mbars + 2, 1); }
  umma_begin(ctl, ncols);
}

// Forward iteration, called by the two CTAs of a cluster (ri = 0, 1) between u2_begin (256 columns of tensor memory)
// and umma_end.  W: fp32 [m][m] (W + eps I is formed where it is read); Wimg: scratch slot for the images of W + eps I;
// Xh: slots 0 .. T-1 receive the images of X_k, slot T X_T in fp32 [m][m]; XTimg: slot that receives the images of X_T
// (for the product Y = X_T M); Ph: slot k receives the images of Q_k.  Returns false if a wait ran out.
__device__ bool ns_forward_umma256(U2Ctx& c, int m, int T, float eps, float alpha_in, const float* W, float* Wimg, float* XTimg,
                                   float* Xh, float* Ph, NsHdr* hdr, float* red, int ri, float& bad) {
  UmmaCtl& ctl = *c.ctl;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64;
  const int gi = ri * 128 + row;                                 // this thread's row in the matrix
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
    if (tid == 0) {               // both CTAs of the cluster arrive at the same values
      float n1; int js;
      norm_argmax(colsum, m, n1, js);                            // near-ties (duplicated landmarks): the lowest index
      red[512] = (alpha_in > 0.f) ? alpha_in : 1.f / (n1 * n1);
      if (ri == 0) {
        hdr->n1 = n1; hdr->ninf = n1; hdr->jstar = js; hdr->istar = js;
        hdr->auto_alpha = !(alpha_in > 0.f);
        hdr->alpha = red[512];
        hdr->pad0 = hdr->pad1 = 0;
      }
    }
    __syncthreads();
  }
  const float alpha = red[512];
  const uint32_t t_acc[2] = {ctl.tmem_base, ctl.tmem_base + 128};
  {  // the images of this CTA's blocks of Wr (not without steps) and of X_0 = alpha Wr^T (without steps also in fp32)
    float v[64];
#pragma unroll 1
    for (int pass = (T == 0 ? 2 : 0); pass < 4; ++pass) {      // passes 0, 1: Wr blocks (ri, 0), (ri, 1); 2, 3: X_0 blocks
      const int ci = pass & 1, gj0 = ci * 128 + col0;
      if (pass < 2) {                                          // a row of W: 128-bit loads where the row allows
#pragma unroll
        for (int q = 0; q < 64; q += 4) {
          if (gi < m && gj0 + q + 3 < m && (m & 3) == 0) {
            const float4 t = *reinterpret_cast<const float4*>(W + (long long)gi * m + gj0 + q);
            v[q] = t.x; v[q + 1] = t.y; v[q + 2] = t.z; v[q + 3] = t.w;
          } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) v[q + u] = (gi < m && gj0 + q + u < m) ? W[(long long)gi * m + gj0 + q + u] : 0.f;
          }
        }
        if (gi < m && gi >= gj0 && gi < gj0 + 64) {
#pragma unroll
          for (int q = 0; q < 64; ++q) if (gi == gj0 + q) v[q] += eps;
        }
      } else {
#pragma unroll
        for (int q = 0; q < 64; ++q) v[q] = (gi < m && gj0 + q < m) ? alpha * (W[(long long)(gj0 + q) * m + gi] + (gi == gj0 + q ? eps : 0.f)) : 0.f;
      }
      if (T == 0) {                                            // X_T = X_0: fp32 to its slot, images to XTimg
        if (gi < m) {
#pragma unroll
          for (int q = 0; q < 64; ++q) if (gj0 + q < m) Xh[(long long)gi * m + gj0 + q] = v[q];
        }
#pragma unroll
        for (int q = 0; q < 64; ++q) bad += isfinite(v[q]) ? 0.f : 1.f;
        u2_store_block(c, v, row, col0, u2_block_w(XTimg, ri, ci), ci, ci == 1);
      } else if (pass < 3) {
        u2_store_block(c, v, row, col0, pass < 2 ? u2_block_w(Wimg, ri, ci) : u2_block_w(Xh, ri, ci), pass, false);
      } else {
        // all three buffers are on their way out: the first must have been read before it is rewritten
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncthreads();
        u2_store_block(c, v, row, col0, u2_block_w(Xh, ri, ci), 0, true);
      }
    }
  }
  phase_sync<kU2Cluster>();
  for (int k = 0; k < T; ++k) {
    const float* X = Xh + (long long)k * kU2Slot;
    float* Q = Ph + (long long)k * kU2Slot;
    {  // Q_k = 2I - Wr X_k
      const U2Group g[2] = {{u2_block(Wimg, ri, 0), true, u2_block(X, 0, 0), u2_block(X, 0, 1), false, t_acc[0], t_acc[1], false},
                            {u2_block(Wimg, ri, 1), true, u2_block(X, 1, 0), u2_block(X, 1, 1), false, t_acc[0], t_acc[1], true}};
      u2_run<2>(c, g, u2_block(X, ri, 0));                      // X_k is complete: its block is fetched beside the epilogue
#pragma unroll 1
      for (int ci = 0; ci < 2; ++ci) {
        const int gj0 = ci * 128 + col0;
        float v[64];
        umma_row<64>(t_acc[ci], col0, v);
#pragma unroll
        for (int q = 0; q < 64; ++q) v[q] = ((gi == gj0 + q && gi < m) ? 2.f : 0.f) - v[q];
        u2_store_block(c, v, row, col0, u2_block_w(Q, ri, ci), ci, ci == 1);
      }
    }
    phase_sync<kU2Cluster>();
    {  // X_{k+1} = X_k Q_k
      const U2Group g[2] = {{u2_block(X, ri, 0), true, u2_block(Q, 0, 0), u2_block(Q, 0, 1), false, t_acc[0], t_acc[1], false},
                            {u2_block(X, ri, 1), true, u2_block(Q, 1, 0), u2_block(Q, 1, 1), false, t_acc[0], t_acc[1], true}};
      u2_run<2>(c, g, k + 1 < T ? u2_block(Wimg, ri, 0) : nullptr);
      float* Xn = Xh + (long long)(k + 1) * kU2Slot;
#pragma unroll 1
      for (int ci = 0; ci < 2; ++ci) {
        const int gj0 = ci * 128 + col0;
        float v[64];
        umma_row<64>(t_acc[ci], col0, v);
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
          u2_store_block(c, v, row, col0, u2_block_w(XTimg, ri, ci), ci, ci == 1);    // and as images, for Y = X_T M
        } else {
          u2_store_block(c, v, row, col0, u2_block_w(Xn, ri, ci), ci, ci == 1);
        }
      }
    }
    phase_sync<kU2Cluster>();
  }
  return c.ok && ctl.timeout == 0;
}

// Y = X_T M on the same engine, between u2_begin and umma_end: M [m][D] (D <= 128, padded with zero columns) becomes two
// block images (one per CTA, slot Mimg), Y[ri] = X_T[ri][0] M[0] + X_T[ri][1] M[1] goes into one accumulator and
// leaves as fp32 rows.  Both CTAs must have passed a cluster barrier since M and the images of X_T were written.
__device__ bool u2_product_y(U2Ctx& c, int m, int D, const float* XTimg, const float* M, float* Mimg, float* Y, int ri) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64, gi = ri * 128 + row;
  const uint32_t t_acc = c.ctl->tmem_base;
  float v[64];
#pragma unroll
  for (int q = 0; q < 64; q += 4) {
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (gi < m && col0 + q < D) t = *reinterpret_cast<const float4*>(M + (long long)gi * D + col0 + q);   // D is a multiple of 4
    v[q] = t.x; v[q + 1] = t.y; v[q + 2] = t.z; v[q + 3] = t.w;
  }
  u2_store_block(c, v, row, col0, u2_block_w(Mimg, 0, ri), 0, true);
  phase_sync<kU2Cluster>();
  const U2Group g[2] = {{u2_block(XTimg, ri, 0), true, u2_block(Mimg, 0, 0), nullptr, false, t_acc, t_acc, false},
                        {u2_block(XTimg, ri, 1), true, u2_block(Mimg, 0, 1), nullptr, false, t_acc, t_acc, true}};
  u2_run<2>(c, g);
  umma_row<64>(t_acc, col0, v);
  if (gi < m) {
#pragma unroll
    for (int q = 0; q < 64; q += 4)
      if (col0 + q < D) *reinterpret_cast<float4*>(Y + (long long)gi * D + col0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
  }
  umma::fence_before_sync();
  __syncthreads();
  return c.ok && c.ctl->timeout == 0;
}

// Adjoint for a symmetric W (same algebra as the 128 x 128 path): per step k, with A = X_k and Q = Q_k as the forward
// pass left them,  H = A^T G,  dW -= H A^T,  G <- G Q^T + Q^T G - 2G.  G0 = dLoss/dX_T, fp32 [m][m].  Scratch slots
// (kU2Slot floats each): Gimg0, Gimg1 (images of G, alternating), Himg, Gpriv.  G is kept in full precision between
// the steps in Gpriv, which only the thread that owns an element reads and writes: laid out [ri][ci][16][256 threads][4]
// so that a warp's accesses are contiguous (a thread's 64 values of a row, read from an [m][m] matrix, would touch 32
// rows per instruction).  Outputs, fp32 [m][m]: Gout = dLoss/dX_0 and dW = -(sum over the steps of H A^T).  Returns
// false if a wait ran out.  Called between u2_begin (512 columns of tensor memory) and umma_end.
__device__ bool ns_backward_umma256(U2Ctx& c, int m, int T, const float* Xh, const float* Ph, const float* G0, float* Gimg0,
                                    float* Gimg1, float* Himg, float* Gpriv, float* Gout, float* dW, int ri) {
  UmmaCtl& ctl = *c.ctl;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64;
  const int gi = ri * 128 + row;
  const bool vec = (m & 3) == 0;
  const uint32_t t_acc[2] = {ctl.tmem_base, ctl.tmem_base + 128}, t_dw[2] = {ctl.tmem_base + 256, ctl.tmem_base + 384};
  // this thread's 64 elements of a block row of an fp32 [m][m] matrix (zero outside)
  auto load_row = [&](const float* src, int gj0, float (&v)[64]) {
#pragma unroll
    for (int q = 0; q < 64; q += 4) {
      if (gi < m && gj0 + q + 3 < m && vec) {
        const float4 t = *reinterpret_cast<const float4*>(src + (long long)gi * m + gj0 + q);
        v[q] = t.x; v[q + 1] = t.y; v[q + 2] = t.z; v[q + 3] = t.w;
      } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) v[q + u] = (gi < m && gj0 + q + u < m) ? src[(long long)gi * m + gj0 + q + u] : 0.f;
      }
    }
  };
  auto store_row = [&](float* dst, int gj0, const float (&v)[64]) {
    if (gi >= m) return;
#pragma unroll
    for (int q = 0; q < 64; q += 4) {
      if (gj0 + q + 3 < m && vec) *reinterpret_cast<float4*>(dst + (long long)gi * m + gj0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
      else {
#pragma unroll
        for (int u = 0; u < 4; ++u) if (gj0 + q + u < m) dst[(long long)gi * m + gj0 + q + u] = v[q + u];
      }
    }
  };
  auto priv = [&](int ci, int q4) { return reinterpret_cast<float4*>(Gpriv) + ((long long)((ri * 2 + ci) * 16 + q4) * 256 + tid); };
  float* Gcur = Gimg0; float* Gnext = Gimg1;
#pragma unroll 1
  for (int ci = 0; ci < 2; ++ci) {           // G in full precision to the private copy (or straight to Gout), its images to Gcur
    float v[64];
    load_row(G0, ci * 128 + col0, v);
    if (T == 0) store_row(Gout, ci * 128 + col0, v);
    else {
#pragma unroll
      for (int q4 = 0; q4 < 16; ++q4) *priv(ci, q4) = make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
      u2_store_block(c, v, row, col0, u2_block_w(Gcur, ri, ci), ci, ci == 1);
    }
  }
  phase_sync<kU2Cluster>();
  for (int k = T - 1; k >= 0; --k) {
    const float* A = Xh + (long long)k * kU2Slot;
    const float* Q = Ph + (long long)k * kU2Slot;
    {  // H = A^T G:  H[ri][ci] = sum_kb (A[kb][ri])^T G[kb][ci]
      const U2Group g[2] = {{u2_block(A, 0, ri), false, u2_block(Gcur, 0, 0), u2_block(Gcur, 0, 1), false, t_acc[0], t_acc[1], false},
                            {u2_block(A, 1, ri), false, u2_block(Gcur, 1, 0), u2_block(Gcur, 1, 1), false, t_acc[0], t_acc[1], true}};
      u2_run<2>(c, g, u2_block(Q, 0, ri));                      // the history is complete: first S of the next phase
#pragma unroll 1
      for (int ci = 0; ci < 2; ++ci) {
        float v[64];
        umma_row<64>(t_acc[ci], col0, v);
        u2_store_block(c, v, row, col0, u2_block_w(Himg, ri, ci), ci, ci == 1);
      }
    }
    phase_sync<kU2Cluster>();
    {  // dW accumulators += H A^T;  G Q^T + Q^T G
      const bool acc = k != T - 1;
      // (the groups that read the history come first: their S block can be fetched before H has arrived)
      const U2Group g[6] = {{u2_block(Q, 0, ri), false, u2_block(Gcur, 0, 0), u2_block(Gcur, 0, 1), false, t_acc[0], t_acc[1], false},
                            {u2_block(Q, 1, ri), false, u2_block(Gcur, 1, 0), u2_block(Gcur, 1, 1), false, t_acc[0], t_acc[1], true},
                            {u2_block(Gcur, ri, 0), true, u2_block(Q, 0, 0), u2_block(Q, 1, 0), true, t_acc[0], t_acc[1], true},
                            {u2_block(Gcur, ri, 1), true, u2_block(Q, 0, 1), u2_block(Q, 1, 1), true, t_acc[0], t_acc[1], true},
                            {u2_block(Himg, ri, 0), true, u2_block(A, 0, 0), u2_block(A, 1, 0), true, t_dw[0], t_dw[1], acc},
                            {u2_block(Himg, ri, 1), true, u2_block(A, 0, 1), u2_block(A, 1, 1), true, t_dw[0], t_dw[1], true}};
      u2_run<6>(c, g, k > 0 ? u2_block(Xh + (long long)(k - 1) * kU2Slot, 0, ri) : nullptr);   // A of the next step
#pragma unroll 1
      for (int ci = 0; ci < 2; ++ci) {
        const int gj0 = ci * 128 + col0;
        float v[64], G[64];
#pragma unroll
        for (int q4 = 0; q4 < 16; ++q4) {
          const float4 t = *priv(ci, q4);
          G[4 * q4] = t.x; G[4 * q4 + 1] = t.y; G[4 * q4 + 2] = t.z; G[4 * q4 + 3] = t.w;
        }
        umma_row<64>(t_acc[ci], col0, v);
#pragma unroll
        for (int q = 0; q < 64; ++q) G[q] = (gi < m && gj0 + q < m) ? v[q] - 2.f * G[q] : 0.f;
        if (k > 0) {
#pragma unroll
          for (int q4 = 0; q4 < 16; ++q4) *priv(ci, q4) = make_float4(G[4 * q4], G[4 * q4 + 1], G[4 * q4 + 2], G[4 * q4 + 3]);
          u2_store_block(c, G, row, col0, u2_block_w(Gnext, ri, ci), ci, ci == 1);
        } else {
          store_row(Gout, gj0, G);             // the last step: dLoss/dX_0 in its [m][m] layout
          if (ci == 1) { umma::fence_before_sync(); __syncthreads(); }
        }
      }
    }
    phase_sync<kU2Cluster>();
    float* tsw = Gcur; Gcur = Gnext; Gnext = tsw;
  }
#pragma unroll 1
  for (int ci = 0; ci < 2; ++ci) {
    const int gj0 = ci * 128 + col0;
    float v[64];
    if (T > 0) umma_row<64>(t_dw[ci], col0, v);
#pragma unroll
    for (int q = 0; q < 64; ++q) v[q] = (T > 0) ? -v[q] : 0.f;
    store_row(dW, gj0, v);
  }
  const bool ok = c.ok && ctl.timeout == 0;
  phase_sync<kU2Cluster>();
  return ok;
}

// dX = dY M^T and dM = X_T^T dY in front of the adjoint, on the same engine (between u2_begin with 512 columns and
// umma_end).  dY, M: fp32 [m][D] (D <= 128, padded with zero columns); XT: fp32 [m][m].  Each CTA turns its block rows
// of dY and M and its two blocks of X_T into images (scratch slots S1: dY blocks 0, 1 and M blocks 2, 3; S2: X_T);
// after a cluster barrier  dX[ri][ci] = dY[ri] M[ci]^T  is one group into two accumulators and
// dM[ri] = sum_kb X_T[kb][ri]^T dY[kb]  two one-sided groups into a third.  Results leave as fp32 rows.  Both CTAs must
// have passed a cluster barrier since dY was written; ends with one.
__device__ bool u2_products_dx_dm(U2Ctx& c, int m, int D, const float* dY, const float* M, const float* XT, float* S1, float* S2,
                                  float* dX, float* dM, int ri) {
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = (warp & 3) * 32 + (tid & 31), col0 = (warp >> 2) * 64, gi = ri * 128 + row;
  const uint32_t tb = c.ctl->tmem_base;
  const bool vec = (m & 3) == 0;
  float v[64];
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    if (pass < 2) {                                              // a block row of dY or of M, D columns of it
      const float* src = pass == 0 ? dY : M;
#pragma unroll
      for (int q = 0; q < 64; q += 4) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        if (gi < m && col0 + q < D) t = *reinterpret_cast<const float4*>(src + (long long)gi * D + col0 + q);   // D is a multiple of 4
        v[q] = t.x; v[q + 1] = t.y; v[q + 2] = t.z; v[q + 3] = t.w;
      }
    } else {                                                     // block (ri, pass - 2) of X_T
      const int gj0 = (pass - 2) * 128 + col0;
#pragma unroll
      for (int q = 0; q < 64; q += 4) {
        if (gi < m && gj0 + q + 3 < m && vec) {
          const float4 t = *reinterpret_cast<const float4*>(XT + (long long)gi * m + gj0 + q);
          v[q] = t.x; v[q + 1] = t.y; v[q + 2] = t.z; v[q + 3] = t.w;
        } else {
#pragma unroll
          for (int u = 0; u < 4; ++u) v[q + u] = (gi < m && gj0 + q + u < m) ? XT[(long long)gi * m + gj0 + q + u] : 0.f;
        }
      }
    }
    float* dst = pass == 0 ? u2_block_w(S1, 0, ri) : (pass == 1 ? u2_block_w(S1, 1, ri) : u2_block_w(S2, ri, pass - 2));
    if (pass < 3) {
      u2_store_block(c, v, row, col0, dst, pass, false);
    } else {
      if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // buffer 0 is on its way out
      __syncthreads();
      u2_store_block(c, v, row, col0, dst, 0, true);
    }
  }
  phase_sync<kU2Cluster>();
  const U2Group g[3] = {{u2_block(S1, 0, ri), true, u2_block(S1, 1, 0), u2_block(S1, 1, 1), true, tb, tb + 128, false},
                        {u2_block(S2, 0, ri), false, u2_block(S1, 0, 0), nullptr, false, tb + 256, tb + 256, false},
                        {u2_block(S2, 1, ri), false, u2_block(S1, 0, 1), nullptr, false, tb + 256, tb + 256, true}};
  u2_run<3>(c, g);
#pragma unroll 1
  for (int ci = 0; ci < 2; ++ci) {
    const int gj0 = ci * 128 + col0;
    umma_row<64>(tb + 128 * ci, col0, v);
    if (gi < m) {
#pragma unroll
      for (int q = 0; q < 64; q += 4) {
        if (gj0 + q + 3 < m && vec) *reinterpret_cast<float4*>(dX + (long long)gi * m + gj0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
        else {
#pragma unroll
          for (int u = 0; u < 4; ++u) if (gj0 + q + u < m) dX[(long long)gi * m + gj0 + q + u] = v[q + u];
        }
      }
    }
  }
  umma_row<64>(tb + 256, col0, v);
  if (gi < m) {
#pragma unroll
    for (int q = 0; q < 64; q += 4)
      if (col0 + q < D) *reinterpret_cast<float4*>(dM + (long long)gi * D + col0 + q) = make_float4(v[q], v[q + 1], v[q + 2], v[q + 3]);
  }
  umma::fence_before_sync();
  __syncthreads();
  const bool ok = c.ok && c.ctl->timeout == 0;
  phase_sync<kU2Cluster>();
  return ok;
}

}  // namespace ln
