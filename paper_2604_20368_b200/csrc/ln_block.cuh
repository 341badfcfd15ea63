// The two steps that surround the Nystrom path inside the attention block: the rotary position embedding on Q and
// K (Sec. 5.1) and the depth-wise convolution branch of Attention = Z V + DWC(V) (Eq. 7), with their adjoints.
// All four kernels are bound by memory traffic (one pass over a [B,H,n,d] tensor each).
#pragma once
#include "ln_common.cuh"

namespace ln {

// Rotary embedding: channel pairs (2i, 2i+1) of the token at grid position p = t - prefix rotate by p * base^(-2i/d);
// the prefix tokens are copied.  Angle, sine, cosine and the rotation itself are formed in double and rounded ONCE to
// the storage type: positions reach 5e4, where a single-precision angle is already 3e-3 rad off, and the rotated
// Q and K feed sign(token - landmark) in the backward pass, so a value that rounds to the other bf16 neighbour than
// the correctly rounded one shows up as a flipped sign.  sign = -1 applies the transpose.
// thread = (token, 4 channels = 2 pairs)
template <typename T> __device__ __forceinline__ T from_d(double x);
template <> __device__ __forceinline__ float from_d<float>(double x) { return (float)x; }
template <> __device__ __forceinline__ bf16 from_d<bf16>(double x) { return __double2bfloat16(x); }

template <typename T>
__global__ void __launch_bounds__(256) k_rope(const T* __restrict__ X, T* __restrict__ out, long long rows, int n, int d,
                                             int prefix, double log2_base, double sign) {
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
  const int quads = d / 4;
  if (e >= rows * quads) return;
  const long long row = e / quads;
  const int c = (int)(e % quads) * 4, t = (int)(row % n);
  const float4 v = ld4(X + row * d + c);
  T* o = out + row * d + c;
  if (t < prefix) { st4(o, v); return; }
  const double pos = (double)(t - prefix);
  double s0, c0, s1, c1;
  sincos(pos * exp2(-(double)c / (double)d * log2_base), &s0, &c0);             // pair index i = c / 2: exponent -2i/d = -c/d
  sincos(pos * exp2(-(double)(c + 2) / (double)d * log2_base), &s1, &c1);
  s0 *= sign; s1 *= sign;
  const double a0 = v.x, b0 = v.y, a1 = v.z, b1 = v.w;
  o[0] = from_d<T>(a0 * c0 - b0 * s0);
  o[1] = from_d<T>(a0 * s0 + b0 * c0);
  o[2] = from_d<T>(a1 * c1 - b1 * s1);
  o[3] = from_d<T>(a1 * s1 + b1 * c1);
}

// out[bh][prefix + r gw + q][c] += sum_{a,b} w[h][c][a][b] src[bh][prefix + (r + a - ks/2) gw + (q + b - ks/2)][c]   (flip = 0)
// or the same with the filter flipped in both directions (flip = 1: the adjoint with respect to src).
// thread = (grid token, 4 channels); filters are read through the read-only cache.
template <typename T>
__global__ void __launch_bounds__(256) k_dwc_add(const T* __restrict__ src, const float* __restrict__ w, T* __restrict__ out,
                                                int H, int n, int d, int prefix, int gh, int gw, int ks, int flip) {
  const int bh = blockIdx.y, h = bh % H, quads = d / 4, half = ks / 2;
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
  if (e >= (long long)gh * gw * quads) return;
  const int tok = (int)(e / quads), c = (int)(e % quads) * 4, r = tok / gw, q = tok % gw;
  const T* sh = src + (long long)bh * n * d + c;
  const float* wh = w + ((long long)h * d + c) * ks * ks;
  T* op = out + ((long long)bh * n + prefix + tok) * d + c;
  float4 acc = ld4(op);
  for (int a = 0; a < ks; ++a) {
    const int rr = r + a - half;
    if (rr < 0 || rr >= gh) continue;
    for (int b = 0; b < ks; ++b) {
      const int qq = q + b - half;
      if (qq < 0 || qq >= gw) continue;
      const int tap = flip ? (ks - 1 - a) * ks + (ks - 1 - b) : a * ks + b;
      const float4 v = ld4(sh + (long long)(prefix + rr * gw + qq) * d);
      acc.x += __ldg(wh + tap) * v.x;
      acc.y += __ldg(wh + ks * ks + tap) * v.y;
      acc.z += __ldg(wh + 2 * ks * ks + tap) * v.z;
      acc.w += __ldg(wh + 3 * ks * ks + tap) * v.w;
    }
  }
  st4(op, acc);
}

// Filter gradient, partial over a chunk of grid tokens: part[bh][chunk][c][tap] = sum_{tokens of the chunk}
// dO[token][c] V[neighbour(token, tap)][c].  grid (chunks, BH), block = d threads (thread = channel), ks <= 7.
template <typename T>
__global__ void __launch_bounds__(128) k_dwc_wgrad(const T* __restrict__ V, const T* __restrict__ dO, float* __restrict__ part,
                                                  int n, int d, int prefix, int gh, int gw, int ks, int tpc) {
  const int chunk = blockIdx.x, bh = blockIdx.y, c = threadIdx.x, half = ks / 2;
  if (c >= d) return;
  float acc[49];
#pragma unroll
  for (int t = 0; t < 49; ++t) acc[t] = 0.f;
  const T* Vh = V + (long long)bh * n * d + c;
  const T* Gh = dO + (long long)bh * n * d + c;
  const int t0 = chunk * tpc, t1 = min(gh * gw, t0 + tpc);
  for (int tok = t0; tok < t1; ++tok) {
    const int r = tok / gw, q = tok % gw;
    const float g = to_f(Gh[(long long)(prefix + tok) * d]);
#pragma unroll
    for (int a = 0; a < 7; ++a)
#pragma unroll
      for (int b = 0; b < 7; ++b) {
        if (a < ks && b < ks) {
          const int rr = r + a - half, qq = q + b - half;
          if (rr >= 0 && rr < gh && qq >= 0 && qq < gw) acc[a * 7 + b] += g * to_f(Vh[(long long)(prefix + rr * gw + qq) * d]);
        }
      }
  }
  float* o = part + (((long long)bh * gridDim.x + chunk) * d + c) * ks * ks;
#pragma unroll
  for (int a = 0; a < 7; ++a)
#pragma unroll
    for (int b = 0; b < 7; ++b)
      if (a < ks && b < ks) o[a * ks + b] = acc[a * 7 + b];
}

// dW[h][e] = sum over the batch elements b and the chunks of part[b H + h][chunk][e], in a fixed order; e < d ks ks
__global__ void __launch_bounds__(256) k_dwc_wreduce(const float* __restrict__ part, float* __restrict__ dW, int B, int H, int chunks, int count) {
  const int h = blockIdx.y, e = blockIdx.x * 256 + threadIdx.x;
  if (e >= count) return;
  float s = 0.f;
  for (int b = 0; b < B; ++b)
    for (int k = 0; k < chunks; ++k) s += part[(((long long)(b * H + h)) * chunks + k) * count + e];
  dW[(long long)h * count + e] = s;
}

}  // namespace ln
