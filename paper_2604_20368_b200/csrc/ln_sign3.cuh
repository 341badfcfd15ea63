// Sign pass of the kernel gradient (App. A) with the upstream factor formed in the same kernel on the tensor cores.
//
// For a kernel block A_ij = k(x_i, y_j) (A = C = k(Q, L) or A = R^T = k(K, L)) the chain rule gives the upstream
//     g_ij = dA_ij A_ij / lambda,      dA = U Y^T      (U = dO, Y = Ytilde for C;  U = V, Y = dM for R^T)
// and App. A gives, with sign(0) = 0,
//     rows[i][c]       = - sum_j g_ij sign(x_ic - y_jc)                 (gradient w.r.t. the tokens x)
//     part[tile][j][c] = + sum_{i in tile} g_ij sign(x_ic - y_jc)       (gradient w.r.t. the landmarks y, per token tile)
//
// One CTA = one tile of 8 TG tokens (TG even, 8..16) x one 64-dim slab of one head.
//   1. dA tile [128 x m] = U tile [128 x D] Y^T on tcgen05: the bf16 U tile is exact and copied as a K-major operand
//      image, Y arrives pre-split (bf16 hi + lo images per 64-landmark block, one bulk copy per block on an mbarrier);
//      two MMAs groups per block (U Y_hi, U Y_lo) into 64 TMEM columns per block.  The operand buffers alias the
//      column-partial buffers of step 2, which are not live yet.
//   2. Rounds of 8 landmarks.  At the end of round r the threads pull the dA columns of round r + 1 out of TMEM
//      (lane = token), multiply by the kernel values A (read from global memory one round ahead) and leave g
//      transposed in shared memory, [landmark][token].  In the round itself thread (tc, tt) owns tokens 8 tt .. 8 tt + 7
//      and dims 4 tc .. 4 tc + 3 of the slab: per landmark and dim one saturating multiply-add per token gives the
//      step h = (sign(x - y) + 1) / 2 (the subtraction is folded into it through a per-landmark scale and offset, see
//      fold_pair), and two packed multiply-adds per token PAIR add g h to the row sums (registers, over all
//      landmarks) and to the column sums (over the thread's 8 tokens).  Packing over token pairs takes g straight
//      from the transposed tile, two tokens per 64-bit half of a 128-bit load.  Column sums of the TG token groups
//      meet in shared memory and are added in a fixed order during the next round; sum_j g and sum_i g come from
//      the g tile.  3 FMA-pipe lane-operations per (pair, dim).
// FUSED = false reads a ready-made g from global memory instead (kept for comparison and tests).
#pragma once
#include "ln_common.cuh"
#include "ln_umma.cuh"
#include "ln_gemm_umma.cuh"

namespace ln {

constexpr int S3_RL = 8;          // landmarks per round
constexpr int S3_DS = 64;         // dims per CTA
constexpr int S3_TGMAX = 16;      // token groups per CTA
constexpr int S3_TOK = 8 * S3_TGMAX;
// shared memory (floats)
constexpr int S3_CP = 0;                                            // [2][RL][TGMAX][64] column partials (aliased by the MMA operands)
constexpr int S3_GS = S3_CP + 2 * S3_RL * S3_TGMAX * S3_DS;         // [2][RL][TOK] g, transposed
constexpr int S3_SB = S3_GS + 2 * S3_RL * S3_TOK;                   // [2][RL][2][64] scales and offsets of the landmark values
constexpr int S3_RS = S3_SB + 2 * S3_RL * 2 * S3_DS;                // [TOK] row sums of g
constexpr int S3_CS = S3_RS + S3_TOK;                               // [<= 256] column sums of g
constexpr int S3_KC = S3_CS + 256;                                  // [<= 256][2] batch-whitening coefficients (kappa, cbar) per landmark
constexpr int S3_END = S3_KC + 512;
__host__ __device__ constexpr size_t sign3_smem_bytes() { return sizeof(float) * (size_t)S3_END; }
static_assert((size_t)(128 * 128 + 2 * GU_KB * 128) * sizeof(bf16) <= sizeof(float) * (size_t)(S3_GS - S3_CP),
              "the operand images of the MMA phase fit in the column-partial buffers they alias");

// Scale and offset of every landmark value (see fold_pair): SB[bh][j][0][c] = s, SB[bh][j][1][c] = b.
__global__ void __launch_bounds__(256) k_fold_landmarks(const float* __restrict__ Lm, float* __restrict__ SB, int D, long long count) {
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;     // index into Lm [BH * m][D]
  if (e >= count) return;
  const long long row = e / D; const int c = (int)(e % D);
  float s, b;
  fold_pair(Lm[e], s, b);
  SB[(row * 2) * D + c] = s;
  SB[(row * 2 + 1) * D + c] = b;
}

__device__ __forceinline__ void s3_cp_async16(void* dst_smem, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;      // src-size 0: the 16 bytes are filled with zeros, nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(umma::s32(dst_smem)), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void s3_cp_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// 4 consecutive fp32 columns of this thread's TMEM lane, in two halves: the load is issued early and its registers
// may be used only after s3_tmem_wait4, which names them as read-write operands so that no use can be moved ahead of it.
__device__ __forceinline__ void s3_tmem_issue4(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void s3_tmem_wait4(uint32_t (&r)[4]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]) : : "memory");
}

// NR = column outputs (float2) per thread and round: 1 with 256 threads, 2 with 128 .. 254.
template <typename TO, int D, int NR, bool FUSED>
__global__ void __launch_bounds__(256, 2) k_sign3(const bf16* __restrict__ tok, const float* __restrict__ SB,
                                                  const bf16* __restrict__ U, const bf16* __restrict__ Yimg,
                                                  const float* __restrict__ A, int lda, TO* __restrict__ rows,
                                                  float* __restrict__ part, int n, int m, float inv_lambda, int* dev_status,
                                                  const float* __restrict__ kap /* NULL or [H][m][2] */, int H) {
  extern __shared__ __align__(128) float s3_smem[];
  __shared__ __align__(8) unsigned long long mbar_y, mbar_mma;
  __shared__ uint32_t tmem_base;
  const int TG = blockDim.y, tc = threadIdx.x, tt = threadIdx.y;
  const int tid = tt * 16 + tc, nthr = 16 * TG, TT8 = 8 * TG, warp = tid >> 5, lane = tid & 31, nwarps = nthr >> 5;
  const int tile = blockIdx.x, slab = blockIdx.y, bh = blockIdx.z, ntiles = gridDim.x;
  const int i0 = tile * TT8;
  float* const Cp = s3_smem + S3_CP;
  float* const Gs = s3_smem + S3_GS;
  float* const SBs = s3_smem + S3_SB;
  float* const rowsum = s3_smem + S3_RS;
  float* const colsum = s3_smem + S3_CS;
  const int nrounds = (m + S3_RL - 1) / S3_RL;
  const int nkb = (m + GU_KB - 1) / GU_KB;
  const int ncols = nkb <= 1 ? 64 : (nkb == 2 ? 128 : 256);
  tok += (long long)bh * n * D + slab * S3_DS + 4 * tc;
  rows += (long long)bh * n * D + slab * S3_DS + 4 * tc;
  A += (long long)bh * n * lda;
  SB += (long long)bh * m * 2 * D + slab * S3_DS;
  float* const outp = part + ((long long)bh * ntiles + tile) * m * D + slab * S3_DS;
  bool ok = true;

  // ---- set-up that does not touch the aliased buffers: zero the never-written slots >= TG of the column partials
  // later (they alias the operands); column sums of g
  for (int e = tid; e < nrounds * S3_RL; e += nthr) colsum[e] = 0.f;
  // batch-statistic whitening (Eq. 5-6 in training mode): the kernel block's upstream gains kappa_l (A_il - cbar_l)
  float* const kc = s3_smem + S3_KC;
  if (kap) for (int e = tid; e < 2 * m; e += nthr) kc[e] = kap[(long long)(bh % H) * m * 2 + e];
  if constexpr (!FUSED) __syncthreads();

  // scale / offset tile of round r into buffer r & 1: 8 landmarks x (64 scales, 64 offsets) = 128 pieces of 16 bytes
  auto fetch_sb = [&](int r) {
    if (tid < 128) {
      const int jj = tid >> 4, piece = tid & 15, j = r * S3_RL + jj;         // piece: 0..7 scales, 8..15 offsets (4 floats each... 16 floats)
      // a row of the tile is [s: 64 floats][b: 64 floats] = 32 pieces of 16 bytes; 128 threads take two pieces each
      float* dst = SBs + (r & 1) * (S3_RL * 2 * S3_DS) + jj * (2 * S3_DS);
      const float* src = SB + (long long)j * 2 * D;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int p = piece * 2 + u, half = p >> 4, off = (p & 15) * 4;       // half 0: scales, 1: offsets
        s3_cp_async16(dst + half * S3_DS + off, src + (long long)half * D + off, j < m);
      }
    }
  };

  // ---- this thread's tokens (8 tokens x 4 dims of the slab) as fp32
  float x[8][4];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int i = i0 + tt * 8 + k;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < n) v = ld4(tok + (long long)i * D);
    x[k][0] = v.x; x[k][1] = v.y; x[k][2] = v.z; x[k][3] = v.w;
  }
  fetch_sb(0);

  // ---- producer role: token row = TMEM lane 32 (warp % 4) + lane; landmark half (4 of the round's 8) by warp / 4.
  // With fewer than 8 warps the first warps take both halves of their rows.
  const int prow = 32 * (warp & 3) + lane, pgi = i0 + prow;
  const bool pin = pgi < n && prow < TT8;
  const int phalf0 = warp >> 2;                                      // 0 for warps 0..3, 1 for warps 4..7
  const bool two_halves = (warp < 4) && (warp + 4 >= nwarps);
  const float* arow = A + (long long)(pin ? pgi : 0) * lda;
  float rs = 0.f;                                                    // this thread's share of sum_j g of its token row

  if constexpr (FUSED) {
    // ================= dA tile on the tensor cores
    bf16* sU = reinterpret_cast<bf16*>(s3_smem + S3_CP);             // [128 x D] K-major image
    bf16* sY = sU + 128 * D;                                         // one block: [2 parts][64 x D]
    if (tid == 0) { umma::mbar_init(&mbar_y, 1); umma::mbar_init(&mbar_mma, 1); }
    if (warp == 0) umma::tmem_alloc(&tmem_base, ncols);
    umma::fence_before_sync();
    __syncthreads();
    umma::fence_after_sync();
    const uint32_t tacc = tmem_base;
    constexpr uint32_t YB = 2 * GU_KB * D * 2;                       // bytes of one block (hi + lo)
    const bf16* Yh = Yimg + (long long)bh * nkb * (2 * GU_KB * D);
    if (tid == 0) { umma::mbar_expect_tx(&mbar_y, YB); umma::bulk_load(sY, Yh, YB, &mbar_y); }
    const bf16* Uh = U + (long long)bh * n * D;
    for (int p = tid; p < 128 * (D / 8); p += nthr) {
      const int r = p / (D / 8), c8 = (p % (D / 8)) * 8;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (i0 + r < n && r < TT8) v = *reinterpret_cast<const uint4*>(Uh + (long long)(i0 + r) * D + c8);
      *reinterpret_cast<uint4*>(sU + umma::img(r, c8, D)) = v;
    }
    umma::fence_smem_to_mma();
    __syncthreads();
    if (tid == 0) {
      const uint32_t idesc = umma::instr_desc(GU_KB, false, false);
      uint32_t ph = 0;
      for (int kb = 0; kb < nkb; ++kb) {
        ok &= umma::mbar_wait(&mbar_y, ph);
        umma::fence_after_sync();
#pragma unroll 1
        for (int pt = 0; pt < 2; ++pt)                               // U Y_hi, U Y_lo
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            umma::mma(tacc + kb * GU_KB, umma::operand_desc(sU, D, true, ks), umma::operand_desc(sY + pt * (GU_KB * D), D, true, ks),
                      idesc, !(pt == 0 && ks == 0));
        umma::commit(&mbar_mma);
        ok &= umma::mbar_wait(&mbar_mma, ph);                        // the block buffer has been read: it may be refilled
        ph ^= 1u;
        if (kb + 1 < nkb) {
          umma::mbar_expect_tx(&mbar_y, YB);
          umma::bulk_load(sY, Yh + (long long)(kb + 1) * (2 * GU_KB * D), YB, &mbar_y);
        }
      }
    }
    umma::fence_before_sync();
    __syncthreads();                                                 // all products complete; the operand buffers are free
    umma::fence_after_sync();
  }
  // unused group slots >= TG of the column partials: zero once (the sum over slots is unrolled over all 16)
  for (int e = tid; e < 2 * S3_RL * (S3_TGMAX - TG) * S3_DS; e += nthr) {
    const int row = e / ((S3_TGMAX - TG) * S3_DS), rest = e % ((S3_TGMAX - TG) * S3_DS);
    Cp[row * (S3_TGMAX * S3_DS) + TG * S3_DS + rest] = 0.f;
  }

  // g of round r into buffer r & 1 (this thread's token row, its 4 or 8 landmarks of the round)
  float4 apre[2];                                                    // kernel values of the round to be produced next
  uint32_t dpre[2][4];                                               // its dA columns, on their way out of tensor memory
  auto fetch_d = [&](int r) {
    if constexpr (FUSED) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        if (u == 1 && !two_halves) continue;
        const int l = r * S3_RL + 4 * (u == 0 ? phalf0 : 1);
        s3_tmem_issue4(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)l, dpre[u]);
      }
    }
  };
  auto fetch_a = [&](int r) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      apre[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (u == 1 && !two_halves) continue;
      const int l = r * S3_RL + 4 * (u == 0 ? phalf0 : 1);
      if (pin && l < lda) apre[u] = *reinterpret_cast<const float4*>(arow + l);
    }
  };
  auto produce = [&](int r) {
    float* gd = Gs + (r & 1) * (S3_RL * S3_TOK) + prow;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (u == 1 && !two_halves) continue;
      const int half = (u == 0 ? phalf0 : 1), l = r * S3_RL + 4 * half;
      float g[4] = {apre[u].x, apre[u].y, apre[u].z, apre[u].w};
      if constexpr (FUSED) {
        s3_tmem_wait4(dpre[u]);
        float da[4] = {__uint_as_float(dpre[u][0]), __uint_as_float(dpre[u][1]), __uint_as_float(dpre[u][2]), __uint_as_float(dpre[u][3])};
        if (kap) {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (l + e < m) da[e] = fmaf(kc[2 * (l + e)], g[e] - kc[2 * (l + e) + 1], da[e]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) g[e] *= da[e];
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (l + e >= m) g[e] = 0.f;
        gd[(4 * half + e) * S3_TOK] = g[e];
      }
      rs += (g[0] + g[1]) + (g[2] + g[3]);
    }
  };
  fetch_a(0);
  fetch_d(0);
  produce(0);
  if (nrounds > 1) fetch_a(1);
  s3_cp_async_wait();
  __syncthreads();

  // column outputs of a round: 8 landmarks x 64 dims = 256 float2; thread o takes landmark o / 32, dims 2 (o % 32).
  // A thread's second output may not exist (o >= 256): it then adds up the partials of output 0 and stores nothing.
  int cjj[NR], coff[NR], csrc[NR];
#pragma unroll
  for (int u = 0; u < NR; ++u) {
    const int o = tid + u * nthr, oc = o < S3_RL * 32 ? o : 0;
    cjj[u] = (o < S3_RL * 32) ? (o >> 5) : (1 << 20);
    coff[u] = (oc >> 5) * D + 2 * (oc & 31);
    csrc[u] = (oc >> 5) * (S3_TGMAX * S3_DS) + 2 * (oc & 31);
  }
  f32x2 accR[4][4];                                                  // [token pair][dim]: lo = even token, hi = odd token
#pragma unroll
  for (int kp = 0; kp < 4; ++kp)
#pragma unroll
    for (int c = 0; c < 4; ++c) accR[kp][c] = 0ull;

  for (int r = 0; r < nrounds; ++r) {
    const int buf = r & 1;
    if (r + 1 < nrounds) { fetch_sb(r + 1); fetch_d(r + 1); }
    const float* gb = Gs + buf * (S3_RL * S3_TOK) + tt * 8;
    const float* sb = SBs + buf * (S3_RL * 2 * S3_DS) + tc * 4;
    float* cp = Cp + buf * (S3_RL * S3_TGMAX * S3_DS) + tt * S3_DS + tc * 4;
    const float* rsrc = Cp + (buf ^ 1) * (S3_RL * S3_TGMAX * S3_DS);     // partials of the previous round
    const int mleft_prev = m - (r - 1) * S3_RL;                          // landmarks of the previous round (r >= 1)
    float2 pend[NR], pend2[NR];
#pragma unroll
    for (int u = 0; u < NR; ++u) { pend[u] = make_float2(0.f, 0.f); pend2[u] = make_float2(0.f, 0.f); }
    // column sums of this round's g tile: warp w takes landmarks w, w + nwarps, ...
    for (int jj = warp; jj < S3_RL; jj += nwarps) {
      const float* g1 = Gs + buf * (S3_RL * S3_TOK) + jj * S3_TOK;
      float s = (g1[lane] + g1[lane + 32]) + (g1[lane + 64] + g1[lane + 96]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) colsum[r * S3_RL + jj] = s;
    }
#pragma unroll
    for (int jj = 0; jj < S3_RL; ++jj) {
      if ((jj & 1) == 0) {                       // a quarter of the previous round's partial sums (round 0 adds up
#pragma unroll                                   // whatever the buffer holds and stores nothing)
        for (int u = 0; u < NR; ++u) {
            const float* src = rsrc + csrc[u] + (jj * 2) * S3_DS;
            const float2 a0 = *reinterpret_cast<const float2*>(src), a1 = *reinterpret_cast<const float2*>(src + S3_DS);
            const float2 a2 = *reinterpret_cast<const float2*>(src + 2 * S3_DS), a3 = *reinterpret_cast<const float2*>(src + 3 * S3_DS);
            pend[u].x += a0.x; pend[u].y += a0.y; pend2[u].x += a1.x; pend2[u].y += a1.y;
            pend[u].x += a2.x; pend[u].y += a2.y; pend2[u].x += a3.x; pend2[u].y += a3.y;
          }
      }
      const float4 s4 = *reinterpret_cast<const float4*>(sb + jj * (2 * S3_DS));
      const float4 b4 = *reinterpret_cast<const float4*>(sb + jj * (2 * S3_DS) + S3_DS);
      const ulonglong2 ga = *reinterpret_cast<const ulonglong2*>(gb + jj * S3_TOK);
      const ulonglong2 gc = *reinterpret_cast<const ulonglong2*>(gb + jj * S3_TOK + 4);
      const f32x2 gp[4] = {ga.x, ga.y, gc.x, gc.y};                 // (g of tokens 2 kp, 2 kp + 1)
      const float sv[4] = {s4.x, s4.y, s4.z, s4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
      f32x2 cacc[4];
#pragma unroll
      for (int kp = 0; kp < 4; ++kp)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const f32x2 h = sat_fma_pair(x[2 * kp][c], x[2 * kp + 1][c], sv[c], bv[c]);
          accR[kp][c] = fma2(gp[kp], h, accR[kp][c]);
          cacc[c] = kp == 0 ? mul2(gp[kp], h) : fma2(gp[kp], h, cacc[c]);
        }
      float ce[4], co[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) unpack2(cacc[c], ce[c], co[c]);
      *reinterpret_cast<float4*>(cp + jj * (S3_TGMAX * S3_DS)) = make_float4(ce[0] + co[0], ce[1] + co[1], ce[2] + co[2], ce[3] + co[3]);
    }
    if (r > 0) {
      float* dst = outp + (long long)(r - 1) * S3_RL * D;
#pragma unroll
      for (int u = 0; u < NR; ++u)
        if (cjj[u] < mleft_prev) {
          const float cs = colsum[(r - 1) * S3_RL + cjj[u]];
          *reinterpret_cast<float2*>(dst + coff[u]) = make_float2(inv_lambda * (2.f * (pend[u].x + pend2[u].x) - cs),
                                                                  inv_lambda * (2.f * (pend[u].y + pend2[u].y) - cs));
        }
    }
    if (r + 1 < nrounds) {
      produce(r + 1);
      if (r + 2 < nrounds) fetch_a(r + 2);
    }
    s3_cp_async_wait();
    __syncthreads();
  }
  // the last round's partials
  {
    const int rl = nrounds - 1, mleft = m - rl * S3_RL;
    const float* rsrc = Cp + (rl & 1) * (S3_RL * S3_TGMAX * S3_DS);
    float* dst = outp + (long long)rl * S3_RL * D;
#pragma unroll
    for (int u = 0; u < NR; ++u)
      if (cjj[u] < mleft) {
        const float* src = rsrc + csrc[u];
        float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int g = 0; g < S3_TGMAX; g += 2) {
          const float2 a = *reinterpret_cast<const float2*>(src + g * S3_DS), b2 = *reinterpret_cast<const float2*>(src + (g + 1) * S3_DS);
          s0.x += a.x; s0.y += a.y; s1.x += b2.x; s1.y += b2.y;
        }
        const float cs = colsum[rl * S3_RL + cjj[u]];
        *reinterpret_cast<float2*>(dst + coff[u]) = make_float2(inv_lambda * (2.f * (s0.x + s1.x) - cs), inv_lambda * (2.f * (s0.y + s1.y) - cs));
      }
  }
  // row sums of g: the first four warps hold the first landmark half of a row (or both), the others the second half
  if (warp < 4) rowsum[prow] = rs;
  __syncthreads();
  if (warp >= 4) rowsum[prow] += rs;
  __syncthreads();
#pragma unroll
  for (int kp = 0; kp < 4; ++kp) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int k = 2 * kp + e, i = i0 + tt * 8 + k;
      if (i < n) {
        const float gs = rowsum[tt * 8 + k];
        float o[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = inv_lambda * (gs - 2.f * (e == 0 ? lo32(accR[kp][c]) : hi32(accR[kp][c])));
        st4(rows + (long long)i * D, make_float4(o[0], o[1], o[2], o[3]));
      }
    }
  }
  if constexpr (FUSED) {
    umma::fence_before_sync();
    __syncthreads();
    if (warp == 0) umma::tmem_dealloc(tmem_base, ncols);
    if (!ok && dev_status && tid == 0) atomicOr(dev_status + bh, 2);
  }
}

}  // namespace ln
