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

// Table of the rotations: tab[pos][i] = (cos, sin) of pos * base^(-2i/d) in double, pos over the token grid, i over the
// d / 2 channel pairs.  Every head and batch element of a call turns by the same angles, so the double-precision
// sine and cosine are formed once per (position, pair) instead of once per element.
__global__ void __launch_bounds__(256) k_rope_table(double2* __restrict__ tab, long long count, int d, double log2_base) {
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
  if (e >= count) return;
  const int i = (int)(e % (d / 2));
  const double pos = (double)(e / (d / 2));
  double sn, cs;
  sincos(pos * exp2(-(double)(2 * i) / (double)d * log2_base), &sn, &cs);
  tab[e] = make_double2(cs, sn);
}

// A thread owns one (token, channel quad) and walks the heads and batch elements of its share (blockIdx.y): the two table
// entries are read once and stay in registers, so the table costs 1 / (heads per share) of what the tensor does.
template <typename T>
__global__ void __launch_bounds__(256) k_rope(const T* __restrict__ X, T* __restrict__ out, int BH, int hpc, int n, int d,
                                             int prefix, const double2* __restrict__ tab, double sign) {
  const int e = blockIdx.x * 256 + threadIdx.x, quads = d / 4;
  if (e >= n * quads) return;
  const int t = e / quads, c = (e % quads) * 4;
  const int h0 = blockIdx.y * hpc, h1 = min(BH, h0 + hpc);
  const long long off = (long long)t * d + c, hstride = (long long)n * d;
  if (t < prefix) {
    for (int h = h0; h < h1; ++h) st4(out + h * hstride + off, ld4(X + h * hstride + off));
    return;
  }
  const double2* tp = tab + (long long)(t - prefix) * (d / 2) + c / 2;         // pairs c / 2 and c / 2 + 1
  const double2 r0 = tp[0], r1 = tp[1];
  const double c0 = r0.x, s0 = r0.y * sign, c1 = r1.x, s1 = r1.y * sign;
  auto turn = [&](const float4& v, T* o) {
    const double a0 = v.x, b0 = v.y, a1 = v.z, b1 = v.w;
    float4 w;
    w.x = to_f(from_d<T>(a0 * c0 - b0 * s0)); w.y = to_f(from_d<T>(a0 * s0 + b0 * c0));
    w.z = to_f(from_d<T>(a1 * c1 - b1 * s1)); w.w = to_f(from_d<T>(a1 * s1 + b1 * c1));
    st4(o, w);                                                                // already rounded to T: the store converts exactly
  };
  int h = h0;
  for (; h + 3 < h1; h += 4) {                                                // four loads in flight
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = ld4(X + (h + u) * hstride + off);
#pragma unroll
    for (int u = 0; u < 4; ++u) turn(v[u], out + (h + u) * hstride + off);
  }
  for (; h < h1; ++h) turn(ld4(X + h * hstride + off), out + h * hstride + off);
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

// Filter gradient, partial over a chunk of grid tokens and one row a of the filter:
//   part[bh][chunk][c][a ks + b] = sum_{tokens of the chunk} dO[token][c] V[neighbour(token, (a, b))][c].
// grid (chunks, BH, ks); 256 threads = d / 4 channel quads x 1024 / d token lanes: a thread walks the tokens lane,
// lane + lanes, ... of the chunk with the ks taps of its filter row for four channels in registers; the lanes are added
// in a fixed order through shared memory.
template <typename T>
__global__ void __launch_bounds__(256) k_dwc_wgrad(const T* __restrict__ V, const T* __restrict__ dO, float* __restrict__ part,
                                                  int n, int d, int prefix, int gh, int gw, int ks, int tpc) {
  __shared__ float red[256][7][4];
  const int chunk = blockIdx.x, bh = blockIdx.y, a = blockIdx.z, half = ks / 2;
  const int quads = d / 4, lanes = 256 / quads, q = (int)threadIdx.x % quads, tl = (int)threadIdx.x / quads, c = 4 * q;
  float acc[7][4];
#pragma unroll
  for (int b = 0; b < 7; ++b)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[b][e] = 0.f;
  const T* Vh = V + (long long)bh * n * d + c;
  const T* Gh = dO + (long long)bh * n * d + c;
  const int t0 = chunk * tpc, t1 = min(gh * gw, t0 + tpc);
  if (tl < lanes)
    for (int tok = t0 + tl; tok < t1; tok += lanes) {
      const int r = tok / gw, q0 = tok % gw, rr = r + a - half;
      if (rr < 0 || rr >= gh) continue;
      const float4 g = ld4(Gh + (long long)(prefix + tok) * d);
#pragma unroll
      for (int b = 0; b < 7; ++b) {
        const int qq = q0 + b - half;
        if (b < ks && qq >= 0 && qq < gw) {
          const float4 v = ld4(Vh + (long long)(prefix + rr * gw + qq) * d);
          acc[b][0] += g.x * v.x; acc[b][1] += g.y * v.y; acc[b][2] += g.z * v.z; acc[b][3] += g.w * v.w;
        }
      }
    }
#pragma unroll
  for (int b = 0; b < 7; ++b)
#pragma unroll
    for (int e = 0; e < 4; ++e) red[threadIdx.x][b][e] = acc[b][e];
  __syncthreads();
  if (tl == 0) {
    float* o = part + (((long long)bh * gridDim.x + chunk) * d + c) * ks * ks + a * ks;
    for (int b = 0; b < ks; ++b)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float s = 0.f;
        for (int w = 0; w < lanes; ++w) s += red[w * quads + q][b][e];
        o[(long long)e * ks * ks + b] = s;
      }
  }
}

// The same for the common 3 x 3 filter with all nine taps in one CTA (grid (chunks, BH)): the upstream row of a token is
// read once, not once per filter row, and the nine neighbour loads of a token are in flight together; a tap outside the
// grid contributes a zero.
template <typename T>
__global__ void __launch_bounds__(256) k_dwc_wgrad3(const T* __restrict__ V, const T* __restrict__ dO, float* __restrict__ part,
                                                   int n, int d, int prefix, int gh, int gw, int tpc) {
  __shared__ float red[256][9][4];
  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int quads = d / 4, lanes = 256 / quads, q = (int)threadIdx.x % quads, tl = (int)threadIdx.x / quads, c = 4 * q;
  float acc[9][4];
#pragma unroll
  for (int t = 0; t < 9; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;
  const T* Vh = V + (long long)bh * n * d + c;
  const T* Gh = dO + (long long)bh * n * d + c;
  const int t0 = chunk * tpc, t1 = min(gh * gw, t0 + tpc);
  if (tl < lanes)
    for (int tok = t0 + tl; tok < t1; tok += lanes) {
      const int r = tok / gw, q0 = tok % gw;
      const float4 g = ld4(Gh + (long long)(prefix + tok) * d);
      float4 v[9];
#pragma unroll
      for (int t = 0; t < 9; ++t) {
        const int rr = r + t / 3 - 1, qq = q0 + t % 3 - 1;
        v[t] = (rr >= 0 && rr < gh && qq >= 0 && qq < gw) ? ld4(Vh + (long long)(prefix + rr * gw + qq) * d) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int t = 0; t < 9; ++t) {
        acc[t][0] = fmaf(g.x, v[t].x, acc[t][0]); acc[t][1] = fmaf(g.y, v[t].y, acc[t][1]);
        acc[t][2] = fmaf(g.z, v[t].z, acc[t][2]); acc[t][3] = fmaf(g.w, v[t].w, acc[t][3]);
      }
    }
#pragma unroll
  for (int t = 0; t < 9; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) red[threadIdx.x][t][e] = acc[t][e];
  __syncthreads();
  // 36 outputs per channel quad: thread (quad q, lane tl) adds the lanes for outputs tl, tl + lanes, ... in a fixed order
  float* o = part + (((long long)bh * gridDim.x + chunk) * d + c) * 9;
  if (tl < lanes)
    for (int k = tl; k < 36; k += lanes) {
      const int e = k / 9, t = k % 9;
      float sacc = 0.f;
      for (int w = 0; w < lanes; ++w) sacc += red[w * quads + q][t][e];
      o[e * 9 + t] = sacc;
    }
}

// dW[h][e] = sum over the batch elements b and the chunks of part[b H + h][chunk][e]; e < count = d ks ks (a multiple of 4).
// grid (ceil(count / 128), H): warp w of a CTA adds the parts w, w + 8, ... for 128 consecutive elements, the eight warps
// are added in a fixed order.
__global__ void __launch_bounds__(256) k_dwc_wreduce(const float* __restrict__ part, float* __restrict__ dW, int B, int H, int chunks, int count) {
  __shared__ float4 red[8][32];
  const int h = blockIdx.y, w = threadIdx.x >> 5, l = threadIdx.x & 31;
  const int e = (blockIdx.x * 32 + l) * 4, P = B * chunks;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (e < count)
    for (int p = w; p < P; p += 8) {
      const int b = p / chunks, k = p % chunks;
      const float4 v = *reinterpret_cast<const float4*>(part + (((long long)(b * H + h)) * chunks + k) * count + e);
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
  red[w][l] = s;
  __syncthreads();
  if (w == 0 && e < count) {
    float4 t = red[0][l];
#pragma unroll
    for (int k = 1; k < 8; ++k) { t.x += red[k][l].x; t.y += red[k][l].y; t.z += red[k][l].z; t.w += red[k][l].w; }
    *reinterpret_cast<float4*>(dW + (long long)h * count + e) = t;
  }
}

}  // namespace ln
