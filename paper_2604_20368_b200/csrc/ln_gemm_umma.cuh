// O[i][c] = sum_l (E[i][l] - mu[i]) Y[l][c] + ybar[c]  on the 5th-generation tensor cores (tcgen05 + TMEM),
// for the two products of the path that reduce over the landmarks: O = (C - mu) Ytilde + ybar (Alg. 1, Prop. 3)
// and dV = R^T dM.
//
// M = 128 tokens per CTA, N = D dims, K = landmarks in blocks of 64.  A = the E tile, converted in the kernel from
// fp32 to a bf16 hi + lo image (K-major); B = Y, which its producer leaves in global memory already split and
// laid out as operand images per 64-landmark block, so that a block arrives with one bulk copy while the E
// block is being converted.  Three MMAs per product (lo*hi, hi*lo, hi*hi), fp32 accumulation in D columns of
// TMEM, issued by one thread; the epilogue goes TMEM -> registers -> bf16 rows in shared memory -> 16-byte
// coalesced stores.  Two CTAs per SM overlap one tile's conversion and epilogue with the other's MMAs.
#pragma once
#include "ln_mma.cuh"
#include "ln_umma.cuh"

namespace ln {

constexpr int GU_KB = 64;                       // landmarks per block
// floats per 64-landmark block of a split operand image of a [m][D] matrix (hi part, lo part)
__host__ __device__ constexpr int gu_block_floats(int D) { return GU_KB * D; }

// [m][D] fp32 (row-major) -> split images per 64-row block: block kb holds rows 64 kb .. 64 kb + 63 as a
// [64][D] image (hi) followed by the same for lo; rows >= m are zero.  Strided over `nthr` threads.
__device__ __forceinline__ void gu_write_images(const float* __restrict__ src, bf16* __restrict__ img, int m, int D,
                                                int t0, int nthr) {
  const int nkb = (m + GU_KB - 1) / GU_KB, per_row = D / 8;
  for (int p = t0; p < nkb * GU_KB * per_row; p += nthr) {
    const int l = p / per_row, c8 = (p % per_row) * 8;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (l < m) { a = *reinterpret_cast<const float4*>(src + (long long)l * D + c8); b = *reinterpret_cast<const float4*>(src + (long long)l * D + c8 + 4); }
    uint2 h0, l0, h1, l1;
    split4(a, h0, l0); split4(b, h1, l1);
    bf16* blk = img + (long long)(l / GU_KB) * (2 * GU_KB * D);
    const int off = umma::img(l % GU_KB, c8, D);
    *reinterpret_cast<uint4*>(blk + off) = make_uint4(h0.x, h0.y, h1.x, h1.y);
    *reinterpret_cast<uint4*>(blk + GU_KB * D + off) = make_uint4(l0.x, l0.y, l1.x, l1.y);
  }
}

// shared memory of k_nn_umma: E block images and Y block images; the bf16 staging of the output tile reuses them
template <int D> __host__ __device__ constexpr size_t nn_umma_smem() { return (size_t)(2 * 128 * GU_KB + 2 * GU_KB * D) * sizeof(bf16); }
// with the convolution branch in the epilogue the output tile is staged in fp32 (one rounding, after the branch is added)
// (behind the staged tile: the head's filters, transposed to [tap][channel], up to 7 x 7 taps)
template <int D> __host__ __device__ constexpr size_t nn_umma_stage_dwc() {
  return nn_umma_smem<D>() > (size_t)128 * (D + 4) * sizeof(float) ? nn_umma_smem<D>() : (size_t)128 * (D + 4) * sizeof(float);
}
template <int D> __host__ __device__ constexpr size_t nn_umma_smem_dwc() { return nn_umma_stage_dwc<D>() + (size_t)49 * D * sizeof(float); }

// one tap of the depth-wise convolution on eight channels: acc += w * v (v: eight bf16 values, w: eight fp32 weights in
// shared memory; a tap outside the grid arrives as zeros)
__device__ __forceinline__ void dwc_tap8(float (&acc)[8], const uint4& v, const float* w) {
  const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
  const float4 w0 = *reinterpret_cast<const float4*>(w), w1 = *reinterpret_cast<const float4*>(w + 4);
  const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    acc[2 * e] = fmaf(wv[2 * e], __uint_as_float(vw[e] << 16), acc[2 * e]);
    acc[2 * e + 1] = fmaf(wv[2 * e + 1], __uint_as_float(vw[e] & 0xffff0000u), acc[2 * e + 1]);
  }
}

// One 128-token tile per CTA; three CTAs per SM hide each other's load latencies.
// DWC: the depth-wise convolution branch of the attention block (Eq. 7) is added in the epilogue, before the one rounding
// to bf16 (O = Z V + DWC(V) in the forward pass; dV = R^T dM + DWC^T(dO) in the backward pass).
template <int D, bool DWC = false>
__global__ void __launch_bounds__(256, 3) k_nn_umma(const float* __restrict__ E, int lde, const float* __restrict__ mu,
                                                    const bf16* __restrict__ Yimg, const float* __restrict__ ybar,
                                                    bf16* __restrict__ O, int n, int m, int* dev_status, DwcEpi epi = DwcEpi()) {
  extern __shared__ __align__(128) unsigned char gu_smem[];
  bf16* sZ = reinterpret_cast<bf16*>(gu_smem);                 // [2][128 * 64]: hi, lo of the E block (K-major image)
  bf16* sY = sZ + 2 * 128 * GU_KB;                             // [2][64 * D]: hi, lo of the Y block (image, rows = K)
  __shared__ unsigned long long mbar_mma, mbar_y;
  __shared__ uint32_t tmem_base;
  const int i0 = blockIdx.x * 128, bh = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int nkb = (m + GU_KB - 1) / GU_KB;
  E += (long long)bh * n * lde;
  O += (long long)bh * n * D;
  if (ybar) ybar += (long long)bh * D;
  Yimg += (long long)bh * nkb * (2 * GU_KB * D);
  if (tid == 0) { umma::mbar_init(&mbar_mma, 1); umma::mbar_init(&mbar_y, 1); }
  if (warp == 0) umma::tmem_alloc(&tmem_base, D);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tacc = tmem_base;
  // E block: thread = (token r of the tile, 32 landmarks of the block)
  const int zr = tid >> 1, zc = (tid & 1) * 32, zi = i0 + zr;
  const bool in = zi < n;
  const float mi = (mu && in) ? mu[(long long)bh * n + zi] : 0.f;
  const uint32_t idesc = umma::instr_desc(D, false, true);
  uint32_t ph_mma = 0, ph_y = 0;
  bool ok = true;
  float4 v[8];                                   // this thread's piece of an E block, fetched one block ahead
  auto fetch = [&](int kb) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int l = kb * GU_KB + zc + 4 * q;
      v[q] = (in && l < m) ? *reinterpret_cast<const float4*>(E + (long long)zi * lde + l) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  fetch(0);
  for (int kb = 0; kb < nkb; ++kb) {
    if (tid == 0) {                              // the Y block arrives while the E block is converted
      umma::mbar_expect_tx(&mbar_y, 2 * GU_KB * D * 2);
      umma::bulk_load(sY, Yimg + (long long)kb * (2 * GU_KB * D), 2 * GU_KB * D * 2, &mbar_y);
    }
#pragma unroll
    for (int q = 0; q < 8; q += 2) {
      float4 a = v[q], b = v[q + 1];
      const int l = kb * GU_KB + zc + 4 * q;
      a.x = (in && l < m) ? a.x - mi : 0.f;     a.y = (in && l + 1 < m) ? a.y - mi : 0.f;
      a.z = (in && l + 2 < m) ? a.z - mi : 0.f; a.w = (in && l + 3 < m) ? a.w - mi : 0.f;
      b.x = (in && l + 4 < m) ? b.x - mi : 0.f; b.y = (in && l + 5 < m) ? b.y - mi : 0.f;
      b.z = (in && l + 6 < m) ? b.z - mi : 0.f; b.w = (in && l + 7 < m) ? b.w - mi : 0.f;
      uint2 h0, l0, h1, l1;
      split4(a, h0, l0); split4(b, h1, l1);
      const int off = umma::img(zr, zc + 4 * q, GU_KB);
      *reinterpret_cast<uint4*>(sZ + off) = make_uint4(h0.x, h0.y, h1.x, h1.y);
      *reinterpret_cast<uint4*>(sZ + 128 * GU_KB + off) = make_uint4(l0.x, l0.y, l1.x, l1.y);
    }
    umma::fence_smem_to_mma();
    __syncthreads();
    if (kb + 1 < nkb) fetch(kb + 1);             // in flight while the MMAs of this block run
    if (tid == 0) {
      ok &= umma::mbar_wait(&mbar_y, ph_y & 1);
      umma::fence_after_sync();
#pragma unroll 1
      for (int part = 0; part < 3; ++part) {     // lo*hi, hi*lo, hi*hi
        const bf16* a = sZ + (part == 0 ? 128 * GU_KB : 0);
        const bf16* b = sY + (part == 1 ? GU_KB * D : 0);
#pragma unroll
        for (int ks = 0; ks < GU_KB / 16; ++ks)
          umma::mma(tacc, umma::operand_desc(a, GU_KB, true, ks), umma::operand_desc(b, D, false, ks), idesc,
                    !(kb == 0 && part == 0 && ks == 0));
      }
      umma::commit(&mbar_mma);
    }
    ph_y ^= 1u;
    ok &= umma::mbar_wait(&mbar_mma, ph_mma & 1);   // the MMAs have read both blocks: the buffers are free again
    ph_mma ^= 1u;
    umma::fence_after_sync();
  }
  // epilogue: thread = (row 32 (warp % 4) + lane, D / 2 columns); rows as bf16 through shared memory (the operand
  // buffers, which no MMA reads any more)
  constexpr int HC = D / 2, LDS_ = D + 8;
  bf16* stage = reinterpret_cast<bf16*>(gu_smem);              // [128][D + 8]
  if constexpr (DWC) {
    constexpr int LDF = D + 4;
    float* fstage = reinterpret_cast<float*>(gu_smem);         // [128][D + 4] fp32
    {
      const int row = (warp & 3) * 32 + (tid & 31), c0 = (warp >> 2) * HC;
#pragma unroll
      for (int cb = 0; cb < HC; cb += 32) {
        float a[32];
        umma::tmem_ld32(umma::tmem_addr(tacc, c0 + cb), a);
#pragma unroll
        for (int q = 0; q < 32; q += 4) {
          const int c = c0 + cb + q;
          float4 o = make_float4(a[q], a[q + 1], a[q + 2], a[q + 3]);
          if (ybar) { o.x += ybar[c]; o.y += ybar[c + 1]; o.z += ybar[c + 2]; o.w += ybar[c + 3]; }
          *reinterpret_cast<float4*>(fstage + row * LDF + c) = o;
        }
      }
    }
    const int kk = epi.ks * epi.ks, half = epi.ks / 2;
    float* wsm = reinterpret_cast<float*>(gu_smem + nn_umma_stage_dwc<D>());     // [tap][D]
    {
      const float* wh = epi.w + (long long)(bh % epi.H) * D * kk;
      for (int e = tid; e < D * kk; e += 256) wsm[(e % kk) * D + e / kk] = wh[e];
    }
    umma::fence_before_sync();
    __syncthreads();
    const bf16* src = static_cast<const bf16*>(epi.src) + (long long)bh * n * D;
    for (int p = tid; p < 128 * (D / 8); p += 256) {
      const int r = p / (D / 8), c8 = (p % (D / 8)) * 8, i = i0 + r;
      if (i >= n) continue;
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = fstage[r * LDF + c8 + e];
      if (i >= epi.prefix) {
        const int tok = i - epi.prefix, gr = tok / epi.gw, gq = tok % epi.gw;
        const bf16* srow = src + (long long)epi.prefix * D + c8;
        if (epi.ks == 3) {                        // the common 3 x 3 filter: all nine loads in flight before the first use
          uint4 v[9];
#pragma unroll
          for (int t = 0; t < 9; ++t) {
            const int rr = gr + t / 3 - 1, qq = gq + t % 3 - 1;
            v[t] = (rr >= 0 && rr < epi.gh && qq >= 0 && qq < epi.gw) ? *reinterpret_cast<const uint4*>(srow + (long long)(rr * epi.gw + qq) * D)
                                                                      : make_uint4(0u, 0u, 0u, 0u);
          }
#pragma unroll
          for (int t = 0; t < 9; ++t) dwc_tap8(acc, v[t], wsm + (epi.flip ? 8 - t : t) * D + c8);
        } else {
          for (int a = 0; a < epi.ks; ++a) {      // a filter row at a time (up to seven loads in flight)
            const int rr = gr + a - half;
            if (rr < 0 || rr >= epi.gh) continue;
            uint4 v[7];
#pragma unroll
            for (int b = 0; b < 7; ++b) {
              const int qq = gq + b - half;
              v[b] = (b < epi.ks && qq >= 0 && qq < epi.gw) ? *reinterpret_cast<const uint4*>(srow + (long long)(rr * epi.gw + qq) * D)
                                                            : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int b = 0; b < 7; ++b)
              if (b < epi.ks) dwc_tap8(acc, v[b], wsm + (epi.flip ? (epi.ks - 1 - a) * epi.ks + (epi.ks - 1 - b) : a * epi.ks + b) * D + c8);
          }
        }
      }
      uint32_t wo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 pr = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
        wo[e] = *reinterpret_cast<const uint32_t*>(&pr);
      }
      *reinterpret_cast<uint4*>(O + (long long)i * D + c8) = make_uint4(wo[0], wo[1], wo[2], wo[3]);
    }
    if (warp == 0) umma::tmem_dealloc(tmem_base, D);
    if (!ok && dev_status && tid == 0) atomicOr(dev_status + bh, 2);
    return;
  }
  {
    const int row = (warp & 3) * 32 + (tid & 31), c0 = (warp >> 2) * HC;
#pragma unroll
    for (int cb = 0; cb < HC; cb += 32) {
      float a[32];
      umma::tmem_ld32(umma::tmem_addr(tacc, c0 + cb), a);
#pragma unroll
      for (int q = 0; q < 32; q += 8) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = c0 + cb + q + 2 * e;
          const float y0 = ybar ? ybar[c] : 0.f, y1 = ybar ? ybar[c + 1] : 0.f;
          const __nv_bfloat162 pr = __floats2bfloat162_rn(a[q + 2 * e] + y0, a[q + 2 * e + 1] + y1);
          w[e] = *reinterpret_cast<const uint32_t*>(&pr);
        }
        *reinterpret_cast<uint4*>(stage + row * LDS_ + c0 + cb + q) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  umma::fence_before_sync();
  __syncthreads();
  for (int p = tid; p < 128 * (D / 8); p += 256) {
    const int r = p / (D / 8), c8 = (p % (D / 8)) * 8;
    if (i0 + r < n) *reinterpret_cast<uint4*>(O + (long long)(i0 + r) * D + c8) = *reinterpret_cast<const uint4*>(stage + r * LDS_ + c8);
  }
  if (warp == 0) umma::tmem_dealloc(tmem_base, D);
  if (!ok && dev_status && tid == 0) atomicOr(dev_status + bh, 2);
}

// =====================================================================================
// G[i][l] = (sum_c U[i][c] Y[l][c]) * E[i][l] / lambda   (the upstream g = dA o A / lambda of a kernel block, App. A)
// M = 128 tokens per CTA, N = 64 landmarks per MMA (one accumulator range of 64 TMEM columns per landmark block),
// K = D.  A = the U tile, bf16 in HBM and therefore exact: copied as it is into a K-major image.  B = Y from the
// same pre-split block images the landmark-reducing product reads (rows = landmarks, so K-major here); two MMAs
// per product (U * Y_hi, U * Y_lo).  Two block buffers: the bulk copy of a block overlaps the MMAs of the other.
// Epilogue per block: TMEM -> registers, times the kernel values (read by row), fp32 rows staged in shared memory,
// coalesced 16-byte stores.
// =====================================================================================
template <int D> __host__ __device__ constexpr size_t ntg_umma_smem() { return (size_t)(128 * D + 2 * 2 * GU_KB * D) * sizeof(bf16); }

template <int D>
__global__ void __launch_bounds__(256, 2) k_ntg_umma(const bf16* __restrict__ U, const bf16* __restrict__ Yimg,
                                                     const float* __restrict__ E, int lde, float* __restrict__ G,
                                                     int n, int m, float inv_lambda, int* dev_status) {
  extern __shared__ __align__(128) unsigned char gu_smem[];
  bf16* sU = reinterpret_cast<bf16*>(gu_smem);                 // [128 x D] K-major image of the U tile
  bf16* sY = sU + 128 * D;                                     // [2 buffers][2 parts][64 * D]
  __shared__ unsigned long long mbar_y[2], mbar_free[2], mbar_done;
  __shared__ uint32_t tmem_base;
  const int i0 = blockIdx.x * 128, bh = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int nkb = (m + GU_KB - 1) / GU_KB;
  const int ncols = nkb <= 1 ? 64 : (nkb == 2 ? 128 : 256);
  U += (long long)bh * n * D;
  E += (long long)bh * n * lde;
  G += (long long)bh * n * lde;
  Yimg += (long long)bh * nkb * (2 * GU_KB * D);
  if (tid == 0) {
    umma::mbar_init(&mbar_y[0], 1); umma::mbar_init(&mbar_y[1], 1);
    umma::mbar_init(&mbar_free[0], 1); umma::mbar_init(&mbar_free[1], 1);
    umma::mbar_init(&mbar_done, 1);
  }
  if (warp == 0) umma::tmem_alloc(&tmem_base, ncols);
  umma::fence_before_sync();
  __syncthreads();
  umma::fence_after_sync();
  const uint32_t tacc = tmem_base;
  constexpr uint32_t YB = 2 * GU_KB * D * 2;     // bytes of one block (hi + lo)
  if (tid == 0)                                  // the first two blocks are on their way while the U tile is copied
    for (int nb = 0; nb < 2 && nb < nkb; ++nb) {
      umma::mbar_expect_tx(&mbar_y[nb], YB);
      umma::bulk_load(sY + nb * (2 * GU_KB * D), Yimg + (long long)nb * (2 * GU_KB * D), YB, &mbar_y[nb]);
    }
  for (int p = tid; p < 128 * (D / 8); p += 256) {
    const int r = p / (D / 8), c8 = (p % (D / 8)) * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (i0 + r < n) v = *reinterpret_cast<const uint4*>(U + (long long)(i0 + r) * D + c8);
    *reinterpret_cast<uint4*>(sU + umma::img(r, c8, D)) = v;
  }
  umma::fence_smem_to_mma();
  __syncthreads();
  // kernel values of the first block for this thread's row, fetched before the products are awaited
  const int row = (warp & 3) * 32 + (tid & 31), ch = (warp >> 2) * 32, gi = i0 + row;
  float4 ev[8];
  auto fetch_e = [&](int nb) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int l = nb * GU_KB + ch + 4 * q;
      ev[q] = (gi < n && l < lde) ? *reinterpret_cast<const float4*>(E + (long long)gi * lde + l) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  fetch_e(0);
  bool ok = true;
  if (tid == 0) {
    const uint32_t idesc = umma::instr_desc(GU_KB, false, false);
    uint32_t ph_y[2] = {0, 0}, ph_f[2] = {0, 0};
    for (int nb = 0; nb < nkb; ++nb) {
      const int b = nb & 1;
      ok &= umma::mbar_wait(&mbar_y[b], ph_y[b] & 1); ph_y[b] ^= 1u;
      umma::fence_after_sync();
      const bf16* yb = sY + b * (2 * GU_KB * D);
#pragma unroll 1
      for (int part = 0; part < 2; ++part)       // U * Y_hi, U * Y_lo
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma::mma(tacc + nb * GU_KB, umma::operand_desc(sU, D, true, ks), umma::operand_desc(yb + part * (GU_KB * D), D, true, ks),
                    idesc, !(part == 0 && ks == 0));
      if (nb + 2 < nkb) {                        // refill this buffer once its MMAs have read it
        umma::commit(&mbar_free[b]);
        ok &= umma::mbar_wait(&mbar_free[b], ph_f[b] & 1); ph_f[b] ^= 1u;
        umma::mbar_expect_tx(&mbar_y[b], YB);
        umma::bulk_load(sY + b * (2 * GU_KB * D), Yimg + (long long)(nb + 2) * (2 * GU_KB * D), YB, &mbar_y[b]);
      }
    }
    umma::commit(&mbar_done);
  }
  ok &= umma::mbar_wait(&mbar_done, 0);
  umma::fence_after_sync();
  // epilogue, one landmark block at a time; the fp32 rows are staged in the (now idle) operand buffers
  constexpr int LDG_ = GU_KB + 4;
  static_assert((size_t)128 * LDG_ * sizeof(float) <= ntg_umma_smem<D>(), "staging fits in the operand buffers");
  float* stage = reinterpret_cast<float*>(gu_smem);             // [128][64 + 4] floats = 34 KB
  for (int nb = 0; nb < nkb; ++nb) {
    float a[32];
    umma::tmem_ld32(umma::tmem_addr(tacc, nb * GU_KB + ch), a);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int l = nb * GU_KB + ch + 4 * q;
      float4 o;
      o.x = (l < m) ? a[4 * q] * ev[q].x * inv_lambda : 0.f;
      o.y = (l + 1 < m) ? a[4 * q + 1] * ev[q].y * inv_lambda : 0.f;
      o.z = (l + 2 < m) ? a[4 * q + 2] * ev[q].z * inv_lambda : 0.f;
      o.w = (l + 3 < m) ? a[4 * q + 3] * ev[q].w * inv_lambda : 0.f;
      *reinterpret_cast<float4*>(stage + row * LDG_ + ch + 4 * q) = o;
    }
    if (nb + 1 < nkb) fetch_e(nb + 1);
    __syncthreads();
    for (int p = tid; p < 128 * (GU_KB / 4); p += 256) {
      const int r = p / (GU_KB / 4), c4 = (p % (GU_KB / 4)) * 4, l = nb * GU_KB + c4;
      if (i0 + r < n && l < lde) *reinterpret_cast<float4*>(G + (long long)(i0 + r) * lde + l) = *reinterpret_cast<const float4*>(stage + r * LDG_ + c4);
    }
    __syncthreads();
  }
  umma::fence_before_sync();
  __syncthreads();
  if (warp == 0) umma::tmem_dealloc(tmem_base, ncols);
  if (!ok && dev_status && tid == 0) atomicOr(dev_status + bh, 2);
}

}  // namespace ln
