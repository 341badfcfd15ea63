// Shared device helpers of the Laplacian-Nystrom kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ln {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// Four consecutive elements as fp32.  The address must be aligned to 4 elements.
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 ld4(const bf16* p) {
  uint2 r = *reinterpret_cast<const uint2*>(p);
  float4 v;
  v.x = __uint_as_float(r.x << 16);
  v.y = __uint_as_float(r.x & 0xffff0000u);
  v.z = __uint_as_float(r.y << 16);
  v.w = __uint_as_float(r.y & 0xffff0000u);
  return v;
}
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void st4(bf16* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = r;
}

// 2^x, approximate (relative error about 2^-22); the exponent of the Laplacian kernel is
// evaluated as 2^(-dist * log2(e) / lambda).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// (sign(t) + 1) / 2 = 0, 1/2, 1 for t < 0, t == 0, t > 0, as one saturating multiply-add on the FMA
// pipe (compare/select instructions would run on the half-rate ALU pipe).  The kernel gradient of
// App. A needs sum_j g_j sign(t_j) = 2 sum_j g_j half_step(t_j) - sum_j g_j, with sign(0) = 0 (the
// appendix states the gradient for t != 0; a tie takes the midpoint sub-gradient).  Exact for every
// |t| >= 2^-101; a smaller non-zero difference is treated as a tie.
__device__ __forceinline__ float half_step(float t) {
  float r;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(t), "f"(1.2676506e30f /* 2^100 */), "f"(0.5f));
  return r;
}

// min(max(a * b + c, 0), 1) in one instruction of the FMA pipe.
__device__ __forceinline__ float sat_fma(float a, float b, float c) {
  float r;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// Scale s and offset b of a threshold y such that sat_fma(x, s, b) = (sign(x - y) + 1) / 2 exactly for every
// bf16 x: s = 2^(22 - exponent(y)), at most 2^126; b = -y s + 1/2 (exact: |y| s < 2^23).
__device__ __forceinline__ void fold_pair(float y, float& s, float& b) {
  const int e = (int)((__float_as_uint(y) >> 23) & 0xffu);
  const int es = e < 23 ? 253 : 276 - e;
  s = __uint_as_float((unsigned)es << 23);
  b = fmaf(-y, s, 0.5f);
}

// Maximum of s[0..m) and the index the gradient of that maximum is taken through: the lowest index whose value lies
// within kNormTie (relative) of the maximum.  Two identical landmarks make two column sums of the landmark kernel
// matrix equal in exact arithmetic; without the window the rounding of the sums would pick the winner (Alg. 2's
// scale depends on the 1- and infinity-norm; any of the tied columns gives a valid subgradient).
constexpr float kNormTie = 1.f / 16384.f;
__device__ __forceinline__ void norm_argmax(const float* s, int m, float& mx, int& idx) {
  mx = -1.f;
  for (int t = 0; t < m; ++t) mx = fmaxf(mx, s[t]);
  const float thr = mx * (1.f - kNormTie);
  idx = 0;
  for (int t = 0; t < m; ++t)
    if (s[t] >= thr) { idx = t; break; }
}

// Packed pair arithmetic (two fp32 lanes per instruction): the FP32 pipe does not get faster, but a
// pair costs one issue slot instead of two, which leaves slots for the shared-memory loads.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 add2(f32x2 x, f32x2 y) { f32x2 z; asm("add.f32x2 %0, %1, %2;" : "=l"(z) : "l"(x), "l"(y)); return z; }
__device__ __forceinline__ f32x2 fma2(f32x2 x, f32x2 y, f32x2 c) { f32x2 z; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(z) : "l"(x), "l"(y), "l"(c)); return z; }
__device__ __forceinline__ f32x2 mul2(f32x2 x, f32x2 y) { f32x2 z; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(z) : "l"(x), "l"(y)); return z; }
// Halves of a pair and a pair from two halves, written as register-pair moves: spelled with 64-bit shifts and ORs the
// compiler emits real integer instructions for them, which cost issue slots in the FP32-bound inner loops.
__device__ __forceinline__ float lo32(f32x2 x) { float a, b; asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(x)); return a; }
__device__ __forceinline__ float hi32(f32x2 x) { float a, b; asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(x)); return b; }
__device__ __forceinline__ f32x2 pack2(float a, float b) { f32x2 z; asm("mov.b64 %0, {%1, %2};" : "=l"(z) : "f"(a), "f"(b)); return z; }
// both halves at once
__device__ __forceinline__ void unpack2(f32x2 x, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(x)); }
// (min(max(x0 s + b, 0), 1), min(max(x1 s + b, 0), 1)) as a pair: two saturating multiply-adds that write the two halves
__device__ __forceinline__ f32x2 sat_fma_pair(float x0, float x1, float s, float b) {
  f32x2 z;
  asm("{\n\t.reg .f32 lo, hi;\n\tfma.rn.sat.f32 lo, %1, %3, %4;\n\tfma.rn.sat.f32 hi, %2, %3, %4;\n\tmov.b64 %0, {lo, hi};\n\t}"
      : "=l"(z) : "f"(x0), "f"(x1), "f"(s), "f"(b));
  return z;
}

// Sum of nparts partial arrays (fixed order p = 0, 1, ...), four consecutive elements at `off`.
// Eight independent loads are issued per batch so that their latencies overlap.
__device__ __forceinline__ float4 sum_parts4(const float* __restrict__ parts, int nparts, long long stride, long long off) {
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  int p = 0;
  for (; p + 8 <= nparts; p += 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = *reinterpret_cast<const float4*>(parts + (long long)(p + u) * stride + off);
#pragma unroll
    for (int u = 0; u < 8; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
  }
  for (; p < nparts; ++p) {
    const float4 v = *reinterpret_cast<const float4*>(parts + (long long)p * stride + off);
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  return s;
}

// Column set a thread owns in a [rows x D] tile worked on by 16 column-threads: DC = D/16
// columns, laid out so that the 16 threads read one contiguous 256-byte (128 for D = 32) run.
template <int D> struct ColMap {
  static constexpr int DC = D / 16;
  // index q in [0, DC) -> column
  __device__ static __forceinline__ int col(int tc, int q) {
    if (D == 32) return tc * 2 + q;
    return (q >> 2) * 64 + tc * 4 + (q & 3);
  }
};

template <int D> __device__ __forceinline__ void ld_cols(const float* row, int tc, float (&v)[D / 16]) {
  if (D == 32) {
    float2 a = *reinterpret_cast<const float2*>(row + tc * 2);
    v[0] = a.x; v[1] = a.y;
  } else {
#pragma unroll
    for (int h = 0; h < D / 64; ++h) {
      float4 a = *reinterpret_cast<const float4*>(row + h * 64 + tc * 4);
      v[h * 4 + 0] = a.x; v[h * 4 + 1] = a.y; v[h * 4 + 2] = a.z; v[h * 4 + 3] = a.w;
    }
  }
}

// Block-wide sum of one float per thread (256 threads); result valid in every thread.
__device__ inline float block_sum(float v, float* red /* >= 8 floats of shared memory */) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float s = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
  __syncthreads();
  return s;
}

// End of a phase of a per-head kernel that CL CTAs of a thread-block cluster share (CL = 1: one CTA per head).
// What the CTAs wrote to global memory before the barrier is visible to all of them after it.  The cluster
// barrier is a hardware barrier (no spinning); every thread of every CTA of the cluster must reach it.
template <int CL> __device__ __forceinline__ void phase_sync() {
  if (CL > 1) {
    __threadfence();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  } else {
    __syncthreads();
  }
}

// Depth-wise convolution branch of the attention block (Eq. 7: Attention = Z V + DWC(V)) as an addition to the output of a
// product kernel: out[bh][prefix + r gw + q][c] += sum_{a,b} w[h][c][a][b] src[bh][prefix + (r+a-ks/2) gw + (q+b-ks/2)][c]
// (zero padding; flip = 1 mirrors the filter, which is the adjoint with respect to src).  src == NULL: nothing is added.
struct DwcEpi { const void* src; const float* w; int H, prefix, gh, gw, ks, flip; };

// Header kept per matrix beside the Newton-Schulz iterates.
struct NsHdr { float alpha, n1, ninf; int jstar, istar, auto_alpha, pad0, pad1; };

// The same columns as ld_cols, as D/32 packed pairs of adjacent dims.
template <int D> __device__ __forceinline__ void ld_col_pairs(const float* row, int tc, f32x2 (&v)[D / 32]) {
  if (D == 32) {
    v[0] = *reinterpret_cast<const f32x2*>(row + tc * 2);
  } else {
#pragma unroll
    for (int h = 0; h < D / 64; ++h) {
      const ulonglong2 a = *reinterpret_cast<const ulonglong2*>(row + h * 64 + tc * 4);
      v[2 * h] = a.x; v[2 * h + 1] = a.y;
    }
  }
}

// acc += g * half_step(t) on a pair of dims: one packed add, two saturating multiply-adds, one packed
// multiply-add (the saturating form has no packed variant).
__device__ __forceinline__ f32x2 sign_step2(f32x2 x, f32x2 neg_y, f32x2 gg, f32x2 acc) {
  const f32x2 t = add2(x, neg_y);
  return fma2(gg, pack2(half_step(lo32(t)), half_step(hi32(t))), acc);
}

}  // namespace ln
