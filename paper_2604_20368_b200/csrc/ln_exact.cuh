// Exact (m = n) Laplacian-kernel attention, forward only: the O(n^2) reference point the Nystrom path approximates
// (Eq. 4 and Eq. 7 with the full kernel matrix G = k(Q, K), never formed in memory):
//     map_mode 1:  O_i = sum_j (G_ij - mu_i) V_j + (1/n) sum_j V_j,   mu_i = (1/n) sum_j G_ij
//     map_mode 0:  O_i = sum_j G_ij V_j
// One CTA = 64 queries; keys and values stream through shared memory in tiles of 64.  Per tile the 64 x 64 kernel
// values are formed on the CUDA cores (subtract, accumulate |.|, one ex2 per pair) and left in shared memory, then
// multiplied into the value tile with fp32 FMAs.  Used for accuracy-against-m curves, not on the training path.
#pragma once
#include "ln_common.cuh"

namespace ln {

template <int D> __host__ __device__ constexpr size_t exact_smem_bytes() { return sizeof(float) * (size_t)(3 * 64 * (D + 4) + 64 * (64 + 4)); }

template <typename T, int D>
__global__ void __launch_bounds__(256) k_exact_fwd(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                                                  T* __restrict__ O, int n, float nscale /* -log2(e) / lambda */, int map_mode) {
  constexpr int P = D + 4, DC = D / 16, GP = 64 + 4;
  extern __shared__ __align__(16) float ex_smem[];
  float* Qs = ex_smem; float* Ks = Qs + 64 * P; float* Vs = Ks + 64 * P; float* Gs = Vs + 64 * P;
  const int i0 = blockIdx.x * 64, bh = blockIdx.y, tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  Q += (long long)bh * n * D; K += (long long)bh * n * D; V += (long long)bh * n * D; O += (long long)bh * n * D;
  for (int idx = tid; idx < 64 * (D / 4); idx += 256) {
    const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + r < n) v = ld4(Q + (long long)(i0 + r) * D + c4);
    *reinterpret_cast<float4*>(Qs + r * P + c4) = v;
  }
  float acc[4][DC], vsum[DC], rs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int q = 0; q < DC; ++q) acc[k][q] = 0.f;
#pragma unroll
  for (int q = 0; q < DC; ++q) vsum[q] = 0.f;
  for (int j0 = 0; j0 < n; j0 += 64) {
    __syncthreads();
    for (int idx = tid; idx < 64 * (D / 4); idx += 256) {
      const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (j0 + r < n) { kv = ld4(K + (long long)(j0 + r) * D + c4); vv = ld4(V + (long long)(j0 + r) * D + c4); }
      *reinterpret_cast<float4*>(Ks + r * P + c4) = kv;
      *reinterpret_cast<float4*>(Vs + r * P + c4) = vv;
    }
    __syncthreads();
    float dist[4][4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) dist[k][q] = 0.f;
#pragma unroll 4
    for (int c = 0; c < D; c += 4) {
      float4 a[4], b[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) a[k] = *reinterpret_cast<const float4*>(Qs + (ty * 4 + k) * P + c);
#pragma unroll
      for (int q = 0; q < 4; ++q) b[q] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * q) * P + c);
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int q = 0; q < 4; ++q)
          dist[k][q] += (fabsf(a[k].x - b[q].x) + fabsf(a[k].y - b[q].y)) + (fabsf(a[k].z - b[q].z) + fabsf(a[k].w - b[q].w));
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float e = (j0 + tx + 16 * q < n) ? ex2(dist[k][q] * nscale) : 0.f;
        Gs[(ty * 4 + k) * GP + tx + 16 * q] = e;
        rs[k] += e;
      }
    __syncthreads();
#pragma unroll 2
    for (int jj = 0; jj < 64; jj += 4) {
      float g[4][4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 t = *reinterpret_cast<const float4*>(Gs + (ty * 4 + k) * GP + jj);
        g[k][0] = t.x; g[k][1] = t.y; g[k][2] = t.z; g[k][3] = t.w;
      }
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        float v[DC];
        ld_cols<D>(Vs + (jj + s) * P, tx, v);
#pragma unroll
        for (int q = 0; q < DC; ++q) vsum[q] += v[q];
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
          for (int q = 0; q < DC; ++q) acc[k][q] = fmaf(g[k][s], v[q], acc[k][q]);
      }
    }
  }
  // row sums over the 16 threads of a query row (lanes tx of a half warp), in a fixed order
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) rs[k] += __shfl_xor_sync(0xffffffffu, rs[k], o);
  const float inv_n = 1.f / (float)n;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = i0 + ty * 4 + k;
    if (i >= n) continue;
#pragma unroll
    for (int q = 0; q < DC; ++q) {
      float o = acc[k][q];
      if (map_mode == 1) o += (inv_n - rs[k] * inv_n) * vsum[q];
      O[(long long)i * D + ColMap<D>::col(tx, q)] = from_f<T>(o);
    }
  }
}

}  // namespace ln
