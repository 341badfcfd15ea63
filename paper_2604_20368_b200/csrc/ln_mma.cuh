// Tensor-core products of the bf16-storage path (warp-level mma.sync m16n8k16, fp32 accumulate).
//
// Every fp32 operand that is produced on the device (kernel values, centred kernel values, the
// folded Y, dM) is split into bf16 hi + bf16 lo and multiplied with two or three MMAs, which
// keeps about 16 mantissa bits: the injective map subtracts a mean that is an order of magnitude
// larger than what is left, so single-bf16 operands would not meet the 2e-2 bar on dQ.
// Operands that are bf16 in HBM already (V, dO) are exact and need no split.
#pragma once
#include "ln_common.cuh"

namespace ln {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* row_ptr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void* row_ptr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// x = hi + lo with hi, lo bf16 (about 16 mantissa bits together)
__device__ __forceinline__ void split2(float x, bf16& hi, bf16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
// four fp32 -> four bf16 hi (packed in uint2) and four bf16 lo
__device__ __forceinline__ void split4(float4 v, uint2& hi, uint2& lo) {
  bf16 h[4], l[4];
  split2(v.x, h[0], l[0]); split2(v.y, h[1], l[1]); split2(v.z, h[2], l[2]); split2(v.w, h[3], l[3]);
  hi.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
  hi.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
  lo.x = (uint32_t)__bfloat16_as_ushort(l[0]) | ((uint32_t)__bfloat16_as_ushort(l[1]) << 16);
  lo.y = (uint32_t)__bfloat16_as_ushort(l[2]) | ((uint32_t)__bfloat16_as_ushort(l[3]) << 16);
}

// Lane's row address for an x4 ldmatrix over a 16x16 block at (r0, c0) of a row-major bf16 tile
// with row stride `ld` elements.  quad_rows: which bit of the 8x8-matrix index moves along rows.
//   A, stored [M][K]        : ldsm_x4   (addr_a (tile, m0, k0))       -> a0..a3
//   A, stored [K][M]        : ldsm_x4_t (addr_at(tile, k0, m0))       -> a0..a3
//   B, stored [N][K]        : ldsm_x4   (addr_b (tile, n0, k0))       -> b0,b1 of n-tile n0 and b0,b1 of n0+8
//   B, stored [K][N]        : ldsm_x4_t (addr_bt(tile, k0, n0))       -> same
__device__ __forceinline__ const bf16* addr_a(const bf16* t, int ld, int m0, int k0) {
  const int lane = threadIdx.x & 31, mat = lane >> 3, r = lane & 7;
  return t + (m0 + r + (mat & 1) * 8) * ld + k0 + (mat >> 1) * 8;
}
__device__ __forceinline__ const bf16* addr_at(const bf16* t, int ld, int k0, int m0) {
  const int lane = threadIdx.x & 31, mat = lane >> 3, r = lane & 7;
  return t + (k0 + r + (mat >> 1) * 8) * ld + m0 + (mat & 1) * 8;
}
__device__ __forceinline__ const bf16* addr_b(const bf16* t, int ld, int n0, int k0) {
  const int lane = threadIdx.x & 31, mat = lane >> 3, r = lane & 7;
  return t + (n0 + r + (mat >> 1) * 8) * ld + k0 + (mat & 1) * 8;
}
__device__ __forceinline__ const bf16* addr_bt(const bf16* t, int ld, int k0, int n0) {
  const int lane = threadIdx.x & 31, mat = lane >> 3, r = lane & 7;
  return t + (k0 + r + (mat & 1) * 8) * ld + n0 + (mat >> 1) * 8;
}

// =====================================================================================
// part[chunk][l][c] = sum_{j in chunk} (E[j][l] - mu[j]) * U[j][c]      (reduction over tokens)
// MMA: M = landmarks, N = dims, K = tokens.  A = E^T from a [token][landmark] tile (transposing
// ldmatrix), split hi/lo; B = U from a [token][dim] bf16 tile (transposing ldmatrix), exact.
// grid (chunks, ceil(m/64), BH); 8 warps = 4 landmark blocks of 16 x 2 halves of the dims.
// =====================================================================================
// The fp32 kernel tile, the bf16 token tile and the row means of a step arrive through a ring of TN_STAGES stages
// filled by 16-byte cp.async copies issued TN_STAGES - 1 steps ahead, so that the loop never waits for global memory;
// the fp32 tile is then centred, split into bf16 hi + lo in a second buffer and multiplied (two MMAs per product).
constexpr int TN_KT = 32;             // tokens per step
constexpr int TN_STAGES = 3;
template <int D> __host__ __device__ constexpr size_t tn_mma_smem() {
  return (size_t)TN_STAGES * (TN_KT * 64 * 4 + TN_KT * (D + 8) * 2 + TN_KT * 4) + 2 * (size_t)TN_KT * (64 + 8) * 2 + (256 / (D / 8)) * D * 4;
}
__device__ __forceinline__ void tn_cp16(void* dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void tn_cp4(void* dst, const void* src, bool valid) {
  const int sz = valid ? 4 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(sz) : "memory");
}

template <int D>
__global__ void __launch_bounds__(256, 3) k_tn_mma(const float* __restrict__ E, int lde, const float* __restrict__ mu,
                                                   const bf16* __restrict__ U, float* __restrict__ part,
                                                   float* __restrict__ colsum_part, int n, int m, int rpc) {
  constexpr int KT = TN_KT, LDE = 64 + 8, LDU = D + 8;
  constexpr int NT = D / 16;        // n8-tiles per warp (half of the dims)
  constexpr int STAGE_BYTES = KT * 64 * 4 + KT * LDU * 2 + KT * 4;
  extern __shared__ __align__(16) unsigned char tn_smem[];
  auto Eraw = [&](int st) { return reinterpret_cast<float*>(tn_smem + (size_t)st * STAGE_BYTES); };                       // [KT][64]
  auto Us = [&](int st) { return reinterpret_cast<bf16*>(tn_smem + (size_t)st * STAGE_BYTES + KT * 64 * 4); };            // [KT][LDU]
  auto Mus = [&](int st) { return reinterpret_cast<float*>(tn_smem + (size_t)st * STAGE_BYTES + KT * 64 * 4 + KT * LDU * 2); };
  bf16* Ehi = reinterpret_cast<bf16*>(tn_smem + (size_t)TN_STAGES * STAGE_BYTES);                                         // [KT][LDE]
  bf16* Elo = Ehi + KT * LDE;
  float* cs_part = reinterpret_cast<float*>(Elo + KT * LDE);                                                              // [256 / (D/8)][D]
  const int chunk = blockIdx.x, l0 = blockIdx.y * 64, bh = blockIdx.z, nchunks = gridDim.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wl = (warp & 3) * 16, wc = (warp >> 2) * (D / 2);
  E += (long long)bh * n * lde;
  U += (long long)bh * n * D;
  if (mu) mu += (long long)bh * n;
  const int jbeg = chunk * rpc, jend = min(n, jbeg + rpc);
  const int nsteps = (jend - jbeg + KT - 1) / KT;
  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[t][q] = 0.f;
  float cs[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) cs[q] = 0.f;
  const bool want_cs = colsum_part != nullptr && blockIdx.y == 0;

  auto issue = [&](int step) {          // copies of step `step` into stage step % TN_STAGES (nothing if past the end)
    if (step < nsteps) {
      const int st = step % TN_STAGES, j0 = jbeg + step * KT;
#pragma unroll
      for (int u = 0; u < 2; ++u) {     // kernel tile: 32 rows x 16 pieces of 4 floats
        const int idx = tid + u * 256, r = idx >> 4, c4 = (idx & 15) * 4, j = j0 + r;
        tn_cp16(Eraw(st) + r * 64 + c4, E + (long long)j * lde + l0 + c4, j < jend && l0 + c4 < lde);
      }
      for (int idx = tid; idx < KT * (D / 8); idx += 256) {   // token tile: 8 bf16 per piece
        const int r = idx / (D / 8), c8 = (idx % (D / 8)) * 8, j = j0 + r;
        tn_cp16(Us(st) + r * LDU + c8, U + (long long)j * D + c8, j < jend);
      }
      if (mu && tid < KT) tn_cp4(Mus(st) + tid, mu + j0 + tid, j0 + tid < jend);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
#pragma unroll
  for (int s0 = 0; s0 < TN_STAGES - 1; ++s0) issue(s0);

  for (int step = 0; step < nsteps; ++step) {
    const int st = step % TN_STAGES, j0 = jbeg + step * KT;
    asm volatile("cp.async.wait_group %0;" ::"n"(TN_STAGES - 2) : "memory");
    __syncthreads();                    // stage `st` has landed for everybody; the MMAs of the previous step have read their buffers
    issue(step + TN_STAGES - 1);        // into the stage the previous step used, which is free now
    {  // centre and split the kernel tile: thread = (token, 8 landmarks)
      const int r = tid >> 3, cb = (tid & 7) * 8, j = j0 + r;
      const float mj = (mu && j < jend) ? Mus(st)[r] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 4) {
        const int l = l0 + cb + k;
        float4 v = *reinterpret_cast<const float4*>(Eraw(st) + r * 64 + cb + k);
        const bool in = j < jend;
        v.x = (in && l < m) ? v.x - mj : 0.f;
        v.y = (in && l + 1 < m) ? v.y - mj : 0.f;
        v.z = (in && l + 2 < m) ? v.z - mj : 0.f;
        v.w = (in && l + 3 < m) ? v.w - mj : 0.f;
        uint2 h, lo;
        split4(v, h, lo);
        *reinterpret_cast<uint2*>(Ehi + r * LDE + cb + k) = h;
        *reinterpret_cast<uint2*>(Elo + r * LDE + cb + k) = lo;
      }
    }
    if (want_cs) {
      for (int idx = tid; idx < KT * (D / 8); idx += 256) {
        const int r = idx / (D / 8), c8 = (idx % (D / 8)) * 8;
        const uint4 v = *reinterpret_cast<const uint4*>(Us(st) + r * LDU + c8);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          cs[2 * q] += __uint_as_float(w[q] << 16);
          cs[2 * q + 1] += __uint_as_float(w[q] & 0xffff0000u);
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int k0 = 0; k0 < KT; k0 += 16) {
      uint32_t ah[4], al[4];
      ldsm_x4_t(ah, addr_at(Ehi, LDE, k0, wl));
      ldsm_x4_t(al, addr_at(Elo, LDE, k0, wl));
#pragma unroll
      for (int t = 0; t < NT; t += 2) {
        uint32_t b[4];
        ldsm_x4_t(b, addr_bt(Us(st), LDU, k0, wc + t * 8));
        mma_bf16(acc[t], ah, b[0], b[1]);
        mma_bf16(acc[t], al, b[0], b[1]);
        mma_bf16(acc[t + 1], ah, b[2], b[3]);
        mma_bf16(acc[t + 1], al, b[2], b[3]);
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  float* out = part + ((long long)bh * nchunks + chunk) * m * D;
  const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    const int c = wc + t * 8 + 2 * t4;
    const int la = l0 + wl + g, lb = la + 8;
    if (la < m) *reinterpret_cast<float2*>(out + (long long)la * D + c) = make_float2(acc[t][0], acc[t][1]);
    if (lb < m) *reinterpret_cast<float2*>(out + (long long)lb * D + c) = make_float2(acc[t][2], acc[t][3]);
  }
  if (colsum_part && blockIdx.y == 0) {   // column sums of U, in a fixed order
    // with 256 threads and D/8 column groups a thread always serves the same group
    const int grp = tid / (D / 8), c8 = (tid % (D / 8)) * 8;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 8; ++q) cs_part[grp * D + c8 + q] = cs[q];
    __syncthreads();
    if (tid < D) {
      float s = 0.f;
      for (int r = 0; r < 256 / (D / 8); ++r) s += cs_part[r * D + tid];
      colsum_part[((long long)bh * nchunks + chunk) * D + tid] = s;
    }
  }
}

// =====================================================================================
// O[i][c] = sum_l (E[i][l] - mu[i]) * Y[l][c] + ybar[c]        (reduction over landmarks)
// MMA: M = tokens, N = dims, K = landmarks.  A from a [token][landmark] tile, B = Y from a
// [landmark][dim] tile (transposing ldmatrix); both split, three MMAs per product.
// grid (ceil(n/64), BH); 8 warps = 4 token blocks of 16 x 2 halves of the dims.
// =====================================================================================
template <int D>
__global__ void __launch_bounds__(256) k_nn_mma(const float* __restrict__ E, int lde, const float* __restrict__ mu,
                                                const float* __restrict__ Y, const float* __restrict__ ybar,
                                                bf16* __restrict__ O, int n, int m) {
  constexpr int KL = 32;            // landmarks per step
  constexpr int LDZ = KL + 8, LDY = D + 8;
  constexpr int NT = D / 16;
  __shared__ __align__(16) bf16 Zhi[64][LDZ];
  __shared__ __align__(16) bf16 Zlo[64][LDZ];
  __shared__ __align__(16) bf16 Yhi[KL][LDY];
  __shared__ __align__(16) bf16 Ylo[KL][LDY];
  const int i0 = blockIdx.x * 64, bh = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wi = (warp & 3) * 16, wc = (warp >> 2) * (D / 2);
  E += (long long)bh * n * lde;
  Y += (long long)bh * m * D;
  O += (long long)bh * n * D;
  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[t][q] = 0.f;

  for (int l0 = 0; l0 < m; l0 += KL) {
    __syncthreads();
    {  // Z tile: 64 tokens x 32 landmarks; thread = (token, 8 landmarks)
      const int r = tid >> 2, cb = (tid & 3) * 8, i = i0 + r;
      const float mi = (mu && i < n) ? mu[(long long)bh * n + i] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 4) {
        const int l = l0 + cb + k;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < n && l < m) {
          v = ld4(E + (long long)i * lde + l);
          v.x = (l < m) ? v.x - mi : 0.f;
          v.y = (l + 1 < m) ? v.y - mi : 0.f;
          v.z = (l + 2 < m) ? v.z - mi : 0.f;
          v.w = (l + 3 < m) ? v.w - mi : 0.f;
        }
        uint2 h, lo;
        split4(v, h, lo);
        *reinterpret_cast<uint2*>(&Zhi[r][cb + k]) = h;
        *reinterpret_cast<uint2*>(&Zlo[r][cb + k]) = lo;
      }
    }
    for (int idx = tid; idx < KL * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4, l = l0 + r;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l < m) v = ld4(Y + (long long)l * D + c4);
      uint2 h, lo;
      split4(v, h, lo);
      *reinterpret_cast<uint2*>(&Yhi[r][c4]) = h;
      *reinterpret_cast<uint2*>(&Ylo[r][c4]) = lo;
    }
    __syncthreads();
#pragma unroll
    for (int k0 = 0; k0 < KL; k0 += 16) {
      uint32_t ah[4], al[4];
      ldsm_x4(ah, addr_a(&Zhi[0][0], LDZ, wi, k0));
      ldsm_x4(al, addr_a(&Zlo[0][0], LDZ, wi, k0));
#pragma unroll
      for (int t = 0; t < NT; t += 2) {
        uint32_t bh4[4], bl4[4];
        ldsm_x4_t(bh4, addr_bt(&Yhi[0][0], LDY, k0, wc + t * 8));
        ldsm_x4_t(bl4, addr_bt(&Ylo[0][0], LDY, k0, wc + t * 8));
        mma_bf16(acc[t], ah, bh4[0], bh4[1]);
        mma_bf16(acc[t], ah, bl4[0], bl4[1]);
        mma_bf16(acc[t], al, bh4[0], bh4[1]);
        mma_bf16(acc[t + 1], ah, bh4[2], bh4[3]);
        mma_bf16(acc[t + 1], ah, bl4[2], bl4[3]);
        mma_bf16(acc[t + 1], al, bh4[2], bh4[3]);
      }
    }
  }
  const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    const int c = wc + t * 8 + 2 * t4;
    const float y0 = ybar ? ybar[(long long)bh * D + c] : 0.f, y1 = ybar ? ybar[(long long)bh * D + c + 1] : 0.f;
    const int ia = i0 + wi + g, ib = ia + 8;
    if (ia < n) *reinterpret_cast<__nv_bfloat162*>(O + (long long)ia * D + c) = __floats2bfloat162_rn(acc[t][0] + y0, acc[t][1] + y1);
    if (ib < n) *reinterpret_cast<__nv_bfloat162*>(O + (long long)ib * D + c) = __floats2bfloat162_rn(acc[t][2] + y0, acc[t][3] + y1);
  }
}

// =====================================================================================
// G[i][l] = (sum_c U[i][c] * Y[l][c]) * E[i][l] / lambda        (reduction over dims)
// MMA: M = tokens, N = landmarks, K = dims.  A = U (bf16 in HBM, exact), B = Y from a
// [landmark][dim] tile (K contiguous), split; two MMAs per product.
// grid (ceil(n/64), ceil(m/64), BH); 8 warps = 4 token blocks of 16 x 2 landmark halves of 32.
// =====================================================================================
template <int D>
__global__ void __launch_bounds__(256) k_nt_g_mma(const bf16* __restrict__ U, const float* __restrict__ Y,
                                                  const float* __restrict__ E, int lde, float* __restrict__ G,
                                                  int n, int m, float inv_lambda) {
  constexpr int DK = (D < 64) ? D : 64;
  constexpr int LD = DK + 8;
  __shared__ __align__(16) bf16 Us[64][LD];
  __shared__ __align__(16) bf16 Yhi[64][LD];
  __shared__ __align__(16) bf16 Ylo[64][LD];
  const int i0 = blockIdx.x * 64, l0 = blockIdx.y * 64, bh = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wi = (warp & 3) * 16, wl = (warp >> 2) * 32;
  U += (long long)bh * n * D;
  Y += (long long)bh * m * D;
  E += (long long)bh * n * lde;
  G += (long long)bh * n * lde;
  float acc[4][4];
#pragma unroll
  for (int t = 0; t < 4; ++t)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[t][q] = 0.f;
  for (int c0 = 0; c0 < D; c0 += DK) {
    __syncthreads();
    for (int idx = tid; idx < 64 * (DK / 8); idx += 256) {
      const int r = idx / (DK / 8), c8 = (idx % (DK / 8)) * 8;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (i0 + r < n) v = *reinterpret_cast<const uint4*>(U + (long long)(i0 + r) * D + c0 + c8);
      *reinterpret_cast<uint4*>(&Us[r][c8]) = v;
    }
    for (int idx = tid; idx < 64 * (DK / 4); idx += 256) {
      const int r = idx / (DK / 4), c4 = (idx % (DK / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l0 + r < m) v = ld4(Y + (long long)(l0 + r) * D + c0 + c4);
      uint2 h, lo;
      split4(v, h, lo);
      *reinterpret_cast<uint2*>(&Yhi[r][c4]) = h;
      *reinterpret_cast<uint2*>(&Ylo[r][c4]) = lo;
    }
    __syncthreads();
#pragma unroll
    for (int k0 = 0; k0 < DK; k0 += 16) {
      uint32_t a[4];
      ldsm_x4(a, addr_a(&Us[0][0], LD, wi, k0));
#pragma unroll
      for (int t = 0; t < 4; t += 2) {
        uint32_t bh4[4], bl4[4];
        ldsm_x4(bh4, addr_b(&Yhi[0][0], LD, wl + t * 8, k0));
        ldsm_x4(bl4, addr_b(&Ylo[0][0], LD, wl + t * 8, k0));
        mma_bf16(acc[t], a, bh4[0], bh4[1]);
        mma_bf16(acc[t], a, bl4[0], bl4[1]);
        mma_bf16(acc[t + 1], a, bh4[2], bh4[3]);
        mma_bf16(acc[t + 1], a, bl4[2], bl4[3]);
      }
    }
  }
  const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int l = l0 + wl + t * 8 + 2 * t4;      // even; lde is a multiple of 4, so l + 1 < lde whenever l < lde
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      const int i = i0 + wi + g + hrow * 8;
      if (i >= n || l >= lde) continue;
      const float2 e = *reinterpret_cast<const float2*>(E + (long long)i * lde + l);
      float2 o;
      o.x = (l < m) ? acc[t][2 * hrow] * e.x * inv_lambda : 0.f;
      o.y = (l + 1 < m) ? acc[t][2 * hrow + 1] * e.y * inv_lambda : 0.f;
      *reinterpret_cast<float2*>(G + (long long)i * lde + l) = o;
    }
  }
}

// =====================================================================================
// Whole-CTA GEMM on global (L2-resident) row-major fp32 matrices with tensor cores:
//   C = beta * Cin + alpha * op(A) op(B) (+ diag on the diagonal),  op(A) is M x K, op(B) is K x N.
// Operands are staged in K-chunks of 32 through shared memory in their stored orientation, split
// into bf16 hi + lo on the way in (three MMAs per product: hi*hi, hi*lo, lo*hi), accumulated in
// fp32 registers.  The next chunk is fetched into registers while the current one is multiplied.
// Executed by all 256 threads (8 warps = 4 row blocks of 16 x 2 column halves of 32 per 64 x 64
// output tile); ends with __syncthreads().  Cin may equal C.
// =====================================================================================
struct __align__(16) MmaGemmSmem {
  bf16 Ah[2560], Al[2560], Bh[2560], Bl[2560];   // [64][40] or [32][72] bf16
};

// Stage geometry: "row-chunk" form = 64 rows x 32 cols ([64][40]); "col-chunk" form = 32 rows x 64 cols ([32][72]).
// 8 floats per thread: thread -> (row, 8 consecutive columns).
template <bool WIDE>   // WIDE: 32 x 64 (col-chunk), else 64 x 32 (row-chunk)
__device__ __forceinline__ void gemm_fetch(const float* src, int ld, int r0, int c0, int rmax, int cmax, float (&v)[8]) {
  const int tid = threadIdx.x;
  const int r = WIDE ? (tid >> 3) : (tid >> 2);
  const int c = WIDE ? (tid & 7) * 8 : (tid & 3) * 8;
  const int gr = r0 + r, gc = c0 + c;
  const float* p = src + (long long)gr * ld + gc;
  if (gr < rmax && gc + 7 < cmax && (ld & 3) == 0 && (gc & 3) == 0) {
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = (gr < rmax && gc + q < cmax) ? p[q] : 0.f;
  }
}
template <bool WIDE>
__device__ __forceinline__ void gemm_stash(bf16* hi, bf16* lo, const float (&v)[8]) {
  const int tid = threadIdx.x;
  const int r = WIDE ? (tid >> 3) : (tid >> 2);
  const int c = WIDE ? (tid & 7) * 8 : (tid & 3) * 8;
  constexpr int LD = WIDE ? 72 : 40;
  uint2 h0, l0, h1, l1;
  split4(make_float4(v[0], v[1], v[2], v[3]), h0, l0);
  split4(make_float4(v[4], v[5], v[6], v[7]), h1, l1);
  *reinterpret_cast<uint4*>(hi + r * LD + c) = make_uint4(h0.x, h0.y, h1.x, h1.y);
  *reinterpret_cast<uint4*>(lo + r * LD + c) = make_uint4(l0.x, l0.y, l1.x, l1.y);
}

template <bool TRA, bool TRB>
__device__ void cta_gemm_mma(int M, int N, int K, const float* A, int lda, const float* Bm, int ldb, float* C,
                             int ldc, float alpha, float beta, const float* Cin, float diag, MmaGemmSmem& sm,
                             int part = 0, int nparts = 1) {
  // part / nparts: this CTA computes the output tiles whose running number is part modulo nparts (the CTAs of a
  // cluster share one product)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = (warp & 3) * 16, wn = (warp >> 2) * 32;
  const int g = lane >> 2, t4 = lane & 3;
  int tile_no = 0;
  for (int i0 = 0; i0 < M; i0 += 64)
    for (int j0 = 0; j0 < N; j0 += 64) {
      if ((tile_no++) % nparts != part) continue;
      float acc[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[t][q] = 0.f;
      float va[8], vb[8];
      // op(A) = A: stored [M][K] -> row-chunk form; op(A) = A^T: stored [K][M] -> col-chunk form
      if (TRA) gemm_fetch<true>(A, lda, 0, i0, K, M, va); else gemm_fetch<false>(A, lda, i0, 0, M, K, va);
      // op(B) = B: stored [K][N] -> col-chunk form; op(B) = B^T: stored [N][K] -> row-chunk form
      if (TRB) gemm_fetch<false>(Bm, ldb, j0, 0, N, K, vb); else gemm_fetch<true>(Bm, ldb, 0, j0, K, N, vb);
      for (int k0 = 0; k0 < K; k0 += 32) {
        __syncthreads();
        gemm_stash<TRA>(sm.Ah, sm.Al, va);
        gemm_stash<!TRB>(sm.Bh, sm.Bl, vb);
        __syncthreads();
        if (k0 + 32 < K) {
          if (TRA) gemm_fetch<true>(A, lda, k0 + 32, i0, K, M, va); else gemm_fetch<false>(A, lda, i0, k0 + 32, M, K, va);
          if (TRB) gemm_fetch<false>(Bm, ldb, j0, k0 + 32, N, K, vb); else gemm_fetch<true>(Bm, ldb, k0 + 32, j0, K, N, vb);
        }
#pragma unroll
        for (int kk = 0; kk < 32; kk += 16) {
          uint32_t ah[4], al[4];
          if (TRA) { ldsm_x4_t(ah, addr_at(sm.Ah, 72, kk, wm)); ldsm_x4_t(al, addr_at(sm.Al, 72, kk, wm)); }
          else     { ldsm_x4(ah, addr_a(sm.Ah, 40, wm, kk));    ldsm_x4(al, addr_a(sm.Al, 40, wm, kk)); }
#pragma unroll
          for (int t = 0; t < 4; t += 2) {
            uint32_t bh4[4], bl4[4];
            if (TRB) { ldsm_x4(bh4, addr_b(sm.Bh, 40, wn + t * 8, kk));    ldsm_x4(bl4, addr_b(sm.Bl, 40, wn + t * 8, kk)); }
            else     { ldsm_x4_t(bh4, addr_bt(sm.Bh, 72, kk, wn + t * 8)); ldsm_x4_t(bl4, addr_bt(sm.Bl, 72, kk, wn + t * 8)); }
            mma_bf16(acc[t], al, bh4[0], bh4[1]);
            mma_bf16(acc[t], ah, bl4[0], bl4[1]);
            mma_bf16(acc[t], ah, bh4[0], bh4[1]);
            mma_bf16(acc[t + 1], al, bh4[2], bh4[3]);
            mma_bf16(acc[t + 1], ah, bl4[2], bl4[3]);
            mma_bf16(acc[t + 1], ah, bh4[2], bh4[3]);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int i = i0 + wm + g + (q >> 1) * 8, j = j0 + wn + t * 8 + 2 * t4 + (q & 1);
          if (i < M && j < N) {
            float v = alpha * acc[t][q];
            if (beta != 0.f) v += beta * Cin[(long long)i * ldc + j];
            if (i == j) v += diag;
            C[(long long)i * ldc + j] = v;
          }
        }
    }
  __syncthreads();
}


}  // namespace ln
