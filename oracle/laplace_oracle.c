/*
 * Float64 CPU oracle for Nystrom-approximated Laplacian-kernel attention
 * (LaplacianFormer, arXiv 2604.20368).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA
 * library can be compared with something written straight from the paper.
 * It shares no code, header, table or helper with the CUDA path, and the
 * CUDA path never calls it.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Everything is plain loops in double precision, one head at a time, in the
 * order in which the paper states the steps.  There is no blocking, fusion
 * or reordering; OpenMP is used only to run independent heads side by side.
 *
 * Per head, with Q,K,V in R^{n x d}, landmarks L in R^{m x d}, decay lambda,
 * ridge eps, T Newton-Schulz steps and a diagonal whitening scale s in R^m:
 *
 *   k(x,y) = exp(-||x-y||_1 / lambda)                    (Laplacian kernel, Sec. 1)
 *   L      = average pooling of the keys over the token grid (Sec. 4.2, landmark selection)
 *   C      = k(Q,L)   [n x m]                            (Eq. 8)
 *   W      = k(L,L) + eps*I   [m x m]                    (Eq. 9, Alg. 2 line "add perturbation")
 *   R      = k(L,K)   [m x n]                            (the C^T factor of Alg. 1)
 *   X_0 = alpha*W^T,  X_{k+1} = X_k (2I - W X_k),  X = X_T   (Alg. 2)
 *   M = R V,  Y = X M
 *   mu_i = mean_l C_il,  Z_il = s_l (C_il - mu_i) + 1/m  (Prop. 3, Eq. 11, diagonal whitening Eq. 6)
 *   O = Z Y                                              (Eq. 7 with G replaced by its Nystrom form)
 *
 * Readings taken where the paper is silent or inconsistent (each is listed
 * with its reason in the design notes of this repository):
 *   - one landmark set (pooled keys) serves all three kernel blocks, so W is
 *     symmetric with unit diagonal as Sec. 4.2 says it is;
 *   - alpha = 1/(||W||_1 ||W||_inf): the printed 2/||W||_2 violates the
 *     condition ||I - alpha W W^T|| < 1 that the same paragraph states;
 *   - the result is the T-step iterate, and the backward pass is the exact
 *     adjoint of those T steps including the dependence of alpha on W;
 *   - sign(0) = 0 in the kernel gradient (App. A states it only for t != 0),
 *     and its sign is the appendix's minus, not the introduction's plus;
 *   - pooling is adaptive (bin a covers rows floor(a*gh/mh) .. ceil((a+1)*gh/mh)-1),
 *     which equals r x r / stride r pooling whenever r divides the grid;
 *   - optionally (lm_f32) a pooled landmark is the single-precision value nearest to the
 *     exact mean, so that sign(token - landmark) is decided on the numbers the device holds;
 *   - the depth-wise-convolution landmark selection Sec. 4.2 mentions as an alternative is one
 *     r x r filter per head and channel applied with stride r to the regions average pooling
 *     would average (no bias; the filter with all taps 1/r^2 is average pooling).
 *   - the conjugate-gradient solver of the ablation (Sec. 5.3, Table 4; solver = 1) is the textbook method from
 *     x_0 = 0 for exactly T steps on (W + eps I) Y = M, column by column, and its backward pass differentiates the
 *     linear system it approximates, each adjoint system by the same T-step method (the paper names the solver only).
 *
 * Beside the path, the two steps that surround it inside the attention block (end of this file): the rotary
 * position embedding on Q and K (Sec. 5.1; positions over the flattened token grid, class tokens not rotated) and
 * Attention = Z V + DWC(V) (Eq. 7; one ks x ks zero-padded cross-correlation filter per head and channel).
 *
 * Pins (tests/test_oracle_*.py): hand values, brute force in numpy, the
 * Kac-Murdock-Szego closed-form inverse, the spectral closed form of the
 * unconverged Newton-Schulz iterate, m = n reproducing exact Laplacian
 * attention, rows of Z summing to one, adjoint identities and central finite
 * differences; for conjugate gradients the one-step closed form, every iterate
 * against the Krylov-subspace minimiser from a dense projected solve,
 * termination in m steps against the library's solve.  Parity unpinned: how close the m < n approximation is to
 * exact attention (the paper prints no error figure).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct oracle_problem {
  int32_t B, H, n, d, m;
  double lambda;
  int32_t ns_iters;
  double ridge_eps;
  double ns_alpha;  /* <= 0: alpha = 1/(||W||_1 ||W||_inf); > 0: used as given, no gradient through it */
  int32_t map_mode; /* 0: O = C X R V;  1: injective map of Prop. 3 applied to the rows of C */
  int32_t lm_mode;  /* 0: landmarks given;  1: landmarks = adaptive average pooling of K;  2: of Q (Sec. 4.2 pools the query tensor in one place);
                       3: two landmark sets as Alg. 1 prints them, Lq = pool(Q) and Lk = pool(K): C = k(Q, Lk), W = k(Lq, Lk) (not symmetric), R = k(Lq, K) */
  int32_t prefix, gh, gw, mh, mw; /* lm_mode 1: n = prefix + gh*gw, m = mh*mw */
  int32_t lm_f32;   /* 1: pooled landmarks are rounded to single precision before use (see fwd_single) */
  const double* lm_filter; /* NULL: average pooling.  Else [H][taps][d], taps = (gh/mh)*(gw/mw): the depth-wise convolution
                              landmark selection of Sec. 4.2 (one r x r filter per head and channel, stride r; the grid must
                              divide).  Tap (u,v) of a region is index u*(gw/mw)+v.  lm_mode 1 or 2 only. */
  int32_t solver;   /* 0: Newton-Schulz (Alg. 2), Y = X_T M.  1: conjugate gradients (the solver of the ablation, Sec. 5.3,
                       Table 4): Y = the ns_iters-step CG iterate of (W + eps I) Y = M, see cg_solve.  One landmark set only. */
} oracle_problem;

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Laplacian kernel block, Sec. 1: K_ij = exp(-sum_c |a_ic - b_jc| / lambda)  */
/* ------------------------------------------------------------------------- */
static void l1_block(int na, int nb, int d, const double* A, const double* Bm, double lambda, double* K) {
  for (int i = 0; i < na; ++i)
    for (int j = 0; j < nb; ++j) {
      double dist = 0.0;
      for (int c = 0; c < d; ++c) dist += fabs(A[(size_t)i * d + c] - Bm[(size_t)j * d + c]);
      K[(size_t)i * nb + j] = exp(-dist / lambda);
    }
}

static double sgn(double t) { return (t > 0.0) - (t < 0.0); }

/*
 * Adjoint of l1_block (App. A): dk/dx_c = -(1/lambda) sign(x_c - y_c) k and
 * dk/dy_c = +(1/lambda) sign(x_c - y_c) k, with sign(0) = 0.
 * dA and dB are ACCUMULATED into.
 */
static void l1_block_bwd(int na, int nb, int d, const double* A, const double* Bm, double lambda,
                         const double* K, const double* dK, double* dA, double* dB) {
  for (int i = 0; i < na; ++i)
    for (int j = 0; j < nb; ++j) {
      double g = dK[(size_t)i * nb + j] * K[(size_t)i * nb + j] / lambda;
      for (int c = 0; c < d; ++c) {
        double s = sgn(A[(size_t)i * d + c] - Bm[(size_t)j * d + c]);
        if (dA) dA[(size_t)i * d + c] -= g * s;
        if (dB) dB[(size_t)j * d + c] += g * s;
      }
    }
}

void oracle_l1_kernel(int batch, int na, int nb, int d, const double* A, const double* Bm, double lambda,
                      double* K, double* rowsum) {
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < batch; ++b) {
    double* Kb = K + (size_t)b * na * nb;
    l1_block(na, nb, d, A + (size_t)b * na * d, Bm + (size_t)b * nb * d, lambda, Kb);
    if (rowsum)
      for (int i = 0; i < na; ++i) {
        double s = 0.0;
        for (int j = 0; j < nb; ++j) s += Kb[(size_t)i * nb + j];
        rowsum[(size_t)b * na + i] = s;
      }
  }
}

void oracle_l1_kernel_bwd(int batch, int na, int nb, int d, const double* A, const double* Bm, double lambda,
                          const double* dK, double* dA, double* dB) {
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < batch; ++b) {
    double* K = (double*)malloc(sizeof(double) * (size_t)na * nb);
    const double* Ab = A + (size_t)b * na * d;
    const double* Bb = Bm + (size_t)b * nb * d;
    l1_block(na, nb, d, Ab, Bb, lambda, K);
    double* dAb = dA + (size_t)b * na * d;
    double* dBb = dB + (size_t)b * nb * d;
    memset(dAb, 0, sizeof(double) * (size_t)na * d);
    memset(dBb, 0, sizeof(double) * (size_t)nb * d);
    l1_block_bwd(na, nb, d, Ab, Bb, lambda, K, dK + (size_t)b * na * nb, dAb, dBb);
    free(K);
  }
}

/* ------------------------------------------------------------------------- */
/* Small dense helpers (row-major)                                            */
/* ------------------------------------------------------------------------- */
/* Cm[p x r] = A[p x q] * B[q x r] */
static void matmul(int p, int q, int r, const double* A, const double* Bm, double* Cm) {
  for (int i = 0; i < p; ++i)
    for (int j = 0; j < r; ++j) {
      double s = 0.0;
      for (int k = 0; k < q; ++k) s += A[(size_t)i * q + k] * Bm[(size_t)k * r + j];
      Cm[(size_t)i * r + j] = s;
    }
}
/* Cm[q x r] = A[p x q]^T * B[p x r] */
static void matmul_tn(int p, int q, int r, const double* A, const double* Bm, double* Cm) {
  for (int i = 0; i < q; ++i)
    for (int j = 0; j < r; ++j) {
      double s = 0.0;
      for (int k = 0; k < p; ++k) s += A[(size_t)k * q + i] * Bm[(size_t)k * r + j];
      Cm[(size_t)i * r + j] = s;
    }
}
/* Cm[p x r] = A[p x q] * B[r x q]^T */
static void matmul_nt(int p, int q, int r, const double* A, const double* Bm, double* Cm) {
  for (int i = 0; i < p; ++i)
    for (int j = 0; j < r; ++j) {
      double s = 0.0;
      for (int k = 0; k < q; ++k) s += A[(size_t)i * q + k] * Bm[(size_t)j * q + k];
      Cm[(size_t)i * r + j] = s;
    }
}

/* ------------------------------------------------------------------------- */
/* Newton-Schulz, Alg. 2                                                      */
/* ------------------------------------------------------------------------- */
/* ||W||_1 = max absolute column sum, ||W||_inf = max absolute row sum.  jstar / istar name the column / row the
   gradient of the norm is taken through.  A maximum is not differentiable where two columns attain it, and two
   identical landmarks (duplicated keys) make two column sums equal exactly, so that rounding alone would pick the
   winner.  Reading: among the columns whose sum lies within NORM_TIE (relative) of the maximum the lowest index is
   taken, which is one valid subgradient and does not depend on the order or precision of the summation.  The norm
   itself is the true maximum. */
#define NORM_TIE (1.0 / 16384.0)
static void norms_1_inf(int m, const double* W, double* n1, int* jstar, double* ninf, int* istar) {
  double* cs = (double*)malloc(sizeof(double) * 2 * (size_t)m);
  double* rs = cs + m;
  *n1 = -1.0; *ninf = -1.0; *jstar = 0; *istar = 0;
  for (int j = 0; j < m; ++j) {
    double s = 0.0;
    for (int i = 0; i < m; ++i) s += fabs(W[(size_t)i * m + j]);
    cs[j] = s;
    if (s > *n1) *n1 = s;
  }
  for (int i = 0; i < m; ++i) {
    double s = 0.0;
    for (int j = 0; j < m; ++j) s += fabs(W[(size_t)i * m + j]);
    rs[i] = s;
    if (s > *ninf) *ninf = s;
  }
  for (int j = 0; j < m; ++j) if (cs[j] >= *n1 * (1.0 - NORM_TIE)) { *jstar = j; break; }
  for (int i = 0; i < m; ++i) if (rs[i] >= *ninf * (1.0 - NORM_TIE)) { *istar = i; break; }
  free(cs);
}

/*
 * One matrix.  Win is the kernel matrix before the ridge.  Xhist (may be NULL)
 * receives X_0 .. X_{T-1} ([T, m, m]); X receives X_T.  Returns alpha.
 */
static double ns_single(int m, const double* Win, int T, double eps, double alpha_in, double* X, double* Xhist) {
  size_t mm = (size_t)m * m;
  double* W = (double*)malloc(sizeof(double) * mm);
  double* P = (double*)malloc(sizeof(double) * mm);
  double* Xn = (double*)malloc(sizeof(double) * mm);
  memcpy(W, Win, sizeof(double) * mm);
  for (int i = 0; i < m; ++i) W[(size_t)i * m + i] += eps;           /* W <- W + eps I */
  double alpha = alpha_in;
  if (!(alpha_in > 0.0)) {
    double n1, ninf; int js, is;
    norms_1_inf(m, W, &n1, &js, &ninf, &is);
    alpha = 1.0 / (n1 * ninf);
  }
  for (int i = 0; i < m; ++i)
    for (int j = 0; j < m; ++j) X[(size_t)i * m + j] = alpha * W[(size_t)j * m + i]; /* X_0 = alpha W^T */
  for (int k = 0; k < T; ++k) {
    if (Xhist) memcpy(Xhist + (size_t)k * mm, X, sizeof(double) * mm);
    matmul(m, m, m, W, X, P);                                        /* P = W X_k */
    for (size_t e = 0; e < mm; ++e) P[e] = -P[e];
    for (int i = 0; i < m; ++i) P[(size_t)i * m + i] += 2.0;         /* 2I - W X_k */
    matmul(m, m, m, X, P, Xn);                                       /* X_{k+1} = X_k (2I - W X_k) */
    memcpy(X, Xn, sizeof(double) * mm);
  }
  free(W); free(P); free(Xn);
  return alpha;
}

/*
 * Exact adjoint of ns_single: given dX = dLoss/dX_T returns dW = dLoss/dW (W
 * before the ridge; the ridge is a constant shift).  When alpha was computed
 * from W its dependence on W is differentiated too.
 */
static void ns_single_bwd(int m, const double* Win, int T, double eps, double alpha_in, const double* dX, double* dW) {
  size_t mm = (size_t)m * m;
  double* W = (double*)malloc(sizeof(double) * mm);
  double* X = (double*)malloc(sizeof(double) * mm);
  double* Xh = (double*)malloc(sizeof(double) * mm * (size_t)(T > 0 ? T : 1));
  double* G = (double*)malloc(sizeof(double) * mm);
  double* P = (double*)malloc(sizeof(double) * mm);
  double* H = (double*)malloc(sizeof(double) * mm);
  double* T1 = (double*)malloc(sizeof(double) * mm);
  double* T2 = (double*)malloc(sizeof(double) * mm);
  double alpha = ns_single(m, Win, T, eps, alpha_in, X, Xh);
  memcpy(W, Win, sizeof(double) * mm);
  for (int i = 0; i < m; ++i) W[(size_t)i * m + i] += eps;
  memcpy(G, dX, sizeof(double) * mm);
  memset(dW, 0, sizeof(double) * mm);
  for (int k = T - 1; k >= 0; --k) {
    const double* A = Xh + (size_t)k * mm;      /* X_k;  X_{k+1} = 2A - A P,  P = W A */
    matmul(m, m, m, W, A, P);
    matmul_tn(m, m, m, A, G, H);                /* H = A^T G          (dP = -H) */
    matmul_nt(m, m, m, H, A, T1);               /* dW += dP A^T = -H A^T */
    for (size_t e = 0; e < mm; ++e) dW[e] -= T1[e];
    matmul_nt(m, m, m, G, P, T1);               /* G P^T */
    matmul_tn(m, m, m, W, H, T2);               /* W^T H = (A W)^T G */
    for (size_t e = 0; e < mm; ++e) G[e] = 2.0 * G[e] - T1[e] - T2[e];
  }
  /* X_0 = alpha W^T */
  double dalpha = 0.0;
  for (int i = 0; i < m; ++i)
    for (int j = 0; j < m; ++j) {
      dalpha += G[(size_t)i * m + j] * W[(size_t)j * m + i];
      dW[(size_t)j * m + i] += alpha * G[(size_t)i * m + j];
    }
  if (!(alpha_in > 0.0)) {
    double n1, ninf; int js, is;
    norms_1_inf(m, W, &n1, &js, &ninf, &is);
    /* alpha = 1/(n1 ninf):  d alpha/d n1 = -alpha/n1,  d alpha/d ninf = -alpha/ninf */
    for (int i = 0; i < m; ++i) dW[(size_t)i * m + js] += dalpha * (-alpha / n1) * sgn(W[(size_t)i * m + js]);
    for (int j = 0; j < m; ++j) dW[(size_t)is * m + j] += dalpha * (-alpha / ninf) * sgn(W[(size_t)is * m + j]);
  }
  free(W); free(X); free(Xh); free(G); free(P); free(H); free(T1); free(T2);
}

/* ------------------------------------------------------------------------- */
/* Conjugate gradients (the other solver of Sec. 5.3 / Table 4)              */
/* ------------------------------------------------------------------------- */
/*
 * The paper names the solver and prints nothing else about it, so this is the textbook method (Hestenes-Stiefel) for
 * the symmetric positive definite system (W + eps I) x = b, started from x_0 = 0, run for exactly T steps, one
 * independent solve per column of B [m][d]:
 *     r_0 = b, p_0 = r_0;   a_k = r_k.r_k / p_k.(Wr p_k);   x_{k+1} = x_k + a_k p_k;   r_{k+1} = r_k - a_k Wr p_k;
 *     b_k = r_{k+1}.r_{k+1} / r_k.r_k;   p_{k+1} = r_{k+1} + b_k p_k.
 * A column whose residual is exactly zero, or whose curvature p.(Wr p) is not positive, stops moving.
 */
static void cg_solve(int m, int d, const double* Win, double eps, int T, const double* Bm, double* X) {
  size_t mm = (size_t)m * m;
  double* Wr = (double*)malloc(sizeof(double) * mm);
  double* r = (double*)malloc(sizeof(double) * m);
  double* pv = (double*)malloc(sizeof(double) * m);
  double* q = (double*)malloc(sizeof(double) * m);
  memcpy(Wr, Win, sizeof(double) * mm);
  for (int i = 0; i < m; ++i) Wr[(size_t)i * m + i] += eps;
  for (int c = 0; c < d; ++c) {
    double rr = 0.0;
    for (int i = 0; i < m; ++i) { X[(size_t)i * d + c] = 0.0; r[i] = Bm[(size_t)i * d + c]; pv[i] = r[i]; rr += r[i] * r[i]; }
    for (int k = 0; k < T; ++k) {
      if (rr == 0.0) break;
      double pq = 0.0;
      for (int i = 0; i < m; ++i) {
        double t = 0.0;
        for (int j = 0; j < m; ++j) t += Wr[(size_t)i * m + j] * pv[j];
        q[i] = t; pq += pv[i] * t;
      }
      if (!(pq > 0.0)) break;
      double a = rr / pq, rn = 0.0;
      for (int i = 0; i < m; ++i) { X[(size_t)i * d + c] += a * pv[i]; r[i] -= a * q[i]; rn += r[i] * r[i]; }
      double be = rn / rr;
      for (int i = 0; i < m; ++i) pv[i] = r[i] + be * pv[i];
      rr = rn;
    }
  }
  free(Wr); free(r); free(pv); free(q);
}

/* X [batch][m][d] = T-step CG iterates of (W + eps I) X = B, W [batch][m][m], B [batch][m][d] */
void oracle_cg_solve(int batch, int m, int d, const double* W, double eps, int iters, const double* Bm, double* X) {
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < batch; ++b)
    cg_solve(m, d, W + (size_t)b * m * m, eps, iters, Bm + (size_t)b * m * d, X + (size_t)b * m * d);
}

void oracle_ns_pinv(int batch, int m, const double* W, int iters, double eps, double alpha,
                    double* X, double* Xhist, double* resid, double* alpha_out) {
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < batch; ++b) {
    size_t mm = (size_t)m * m;
    double a = ns_single(m, W + b * mm, iters, eps, alpha, X + b * mm,
                         Xhist ? Xhist + (size_t)b * iters * mm : NULL);
    if (alpha_out) alpha_out[b] = a;
    if (resid) { /* || I - (W + eps I) X_T ||_F */
      double* Wr = (double*)malloc(sizeof(double) * mm);
      double* P = (double*)malloc(sizeof(double) * mm);
      memcpy(Wr, W + b * mm, sizeof(double) * mm);
      for (int i = 0; i < m; ++i) Wr[(size_t)i * m + i] += eps;
      matmul(m, m, m, Wr, X + b * mm, P);
      double s = 0.0;
      for (int i = 0; i < m; ++i)
        for (int j = 0; j < m; ++j) {
          double e = (i == j ? 1.0 : 0.0) - P[(size_t)i * m + j];
          s += e * e;
        }
      resid[b] = sqrt(s);
      free(Wr); free(P);
    }
  }
}

void oracle_ns_pinv_bwd(int batch, int m, const double* W, int iters, double eps, double alpha,
                        const double* dX, double* dW) {
#pragma omp parallel for schedule(dynamic)
  for (int b = 0; b < batch; ++b) {
    size_t mm = (size_t)m * m;
    ns_single_bwd(m, W + b * mm, iters, eps, alpha, dX + b * mm, dW + b * mm);
  }
}

/* ------------------------------------------------------------------------- */
/* Landmark selection by average pooling over the token grid (Sec. 4.2)       */
/* ------------------------------------------------------------------------- */
static int bin_lo(int a, int g, int mbin) { return (int)(((long long)a * g) / mbin); }
static int bin_hi(int a, int g, int mbin) { return (int)((((long long)(a + 1)) * g + mbin - 1) / mbin); }

/* w: NULL, or this head's filter [taps][d] (depth-wise convolution selection, Sec. 4.2) */
static const double* head_filter(const oracle_problem* p, int bh) {
  if (!p->lm_filter) return NULL;
  return p->lm_filter + (size_t)(bh % p->H) * (size_t)((p->gh / p->mh) * (p->gw / p->mw)) * p->d;
}
static void pool_single(const oracle_problem* p, const double* K, double* L, const double* w) {
  int d = p->d;
  if (w) {                         /* L[(a,b)][c] = sum over the taps (u,v) of the region of w[(u,v)][c] K[token][c] */
    int rh = p->gh / p->mh, rw = p->gw / p->mw;
    for (int a = 0; a < p->mh; ++a)
      for (int b = 0; b < p->mw; ++b) {
        double* Ll = L + (size_t)(a * p->mw + b) * d;
        for (int c = 0; c < d; ++c) Ll[c] = 0.0;
        for (int u = 0; u < rh; ++u)
          for (int v = 0; v < rw; ++v) {
            const double* kt = K + (size_t)(p->prefix + (a * rh + u) * p->gw + (b * rw + v)) * d;
            const double* wt = w + (size_t)(u * rw + v) * d;
            for (int c = 0; c < d; ++c) Ll[c] += wt[c] * kt[c];
          }
      }
    return;
  }
  for (int a = 0; a < p->mh; ++a)
    for (int b = 0; b < p->mw; ++b) {
      int r0 = bin_lo(a, p->gh, p->mh), r1 = bin_hi(a, p->gh, p->mh);
      int c0 = bin_lo(b, p->gw, p->mw), c1 = bin_hi(b, p->gw, p->mw);
      double cnt = (double)(r1 - r0) * (double)(c1 - c0);
      double* Ll = L + (size_t)(a * p->mw + b) * d;
      for (int c = 0; c < d; ++c) Ll[c] = 0.0;
      for (int r = r0; r < r1; ++r)
        for (int q = c0; q < c1; ++q) {
          const double* kt = K + (size_t)(p->prefix + r * p->gw + q) * d;
          for (int c = 0; c < d; ++c) Ll[c] += kt[c];
        }
      for (int c = 0; c < d; ++c) Ll[c] /= cnt;
    }
}

/* dK += pool^T(dL); with a filter w also dw += the gradient of the filter (K: the tensor that was pooled) */
static void pool_single_bwd(const oracle_problem* p, const double* dL, double* dK, const double* K, const double* w, double* dw) {
  int d = p->d;
  if (w) {
    int rh = p->gh / p->mh, rw = p->gw / p->mw;
    for (int a = 0; a < p->mh; ++a)
      for (int b = 0; b < p->mw; ++b) {
        const double* dLl = dL + (size_t)(a * p->mw + b) * d;
        for (int u = 0; u < rh; ++u)
          for (int v = 0; v < rw; ++v) {
            size_t tok = (size_t)(p->prefix + (a * rh + u) * p->gw + (b * rw + v)) * d;
            const double* wt = w + (size_t)(u * rw + v) * d;
            for (int c = 0; c < d; ++c) {
              dK[tok + c] += wt[c] * dLl[c];
              if (dw) dw[(size_t)(u * rw + v) * d + c] += dLl[c] * K[tok + c];
            }
          }
      }
    return;
  }
  for (int a = 0; a < p->mh; ++a)
    for (int b = 0; b < p->mw; ++b) {
      int r0 = bin_lo(a, p->gh, p->mh), r1 = bin_hi(a, p->gh, p->mh);
      int c0 = bin_lo(b, p->gw, p->mw), c1 = bin_hi(b, p->gw, p->mw);
      double cnt = (double)(r1 - r0) * (double)(c1 - c0);
      const double* dLl = dL + (size_t)(a * p->mw + b) * d;
      for (int r = r0; r < r1; ++r)
        for (int q = c0; q < c1; ++q) {
          double* kt = dK + (size_t)(p->prefix + r * p->gw + q) * d;
          for (int c = 0; c < d; ++c) kt[c] += dLl[c] / cnt;
        }
    }
}

void oracle_landmarks_pool(const oracle_problem* p, const double* K, double* L) {
  int BH = p->B * p->H;
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < BH; ++h)
    pool_single(p, K + (size_t)h * p->n * p->d, L + (size_t)h * p->m * p->d, head_filter(p, h));
}

/* dK is overwritten with pool^T(dL) */
void oracle_landmarks_pool_bwd(const oracle_problem* p, const double* dL, double* dK) {
  int BH = p->B * p->H;
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < BH; ++h) {
    double* dKh = dK + (size_t)h * p->n * p->d;
    memset(dKh, 0, sizeof(double) * (size_t)p->n * p->d);
    pool_single_bwd(p, dL + (size_t)h * p->m * p->d, dKh, NULL, head_filter(p, h), NULL);
  }
}

/* ------------------------------------------------------------------------- */
/* The whole path for one head                                                */
/* ------------------------------------------------------------------------- */
typedef struct head_ctx {
  double *L, *C, *R, *W, *X, *M, *Y, *Z;
  double *Lq;   /* query-side landmarks of the two-set variant (lm_mode 3); otherwise the same array as L */
  double *Lq_own;
} head_ctx;

static void ctx_alloc(head_ctx* x, int n, int d, int m) {
  x->L = (double*)malloc(sizeof(double) * (size_t)m * d);
  x->Lq_own = (double*)malloc(sizeof(double) * (size_t)m * d);
  x->Lq = x->L;
  x->C = (double*)malloc(sizeof(double) * (size_t)n * m);
  x->R = (double*)malloc(sizeof(double) * (size_t)m * n);
  x->W = (double*)malloc(sizeof(double) * (size_t)m * m);
  x->X = (double*)malloc(sizeof(double) * (size_t)m * m);
  x->M = (double*)malloc(sizeof(double) * (size_t)m * d);
  x->Y = (double*)malloc(sizeof(double) * (size_t)m * d);
  x->Z = (double*)malloc(sizeof(double) * (size_t)n * m);
}
static void ctx_free(head_ctx* x) {
  free(x->L); free(x->Lq_own); free(x->C); free(x->R); free(x->W); free(x->X); free(x->M); free(x->Y); free(x->Z);
}

/* s: whitening scale of this head ([m]) or NULL for ones */
static void fwd_single(const oracle_problem* p, const double* Q, const double* K, const double* V,
                       const double* Lin, const double* s, const double* wf, head_ctx* x, double* O) {
  /* wf: this head's landmark-selection filter (see oracle_problem.lm_filter) or NULL for average pooling */
  int n = p->n, d = p->d, m = p->m;
  if (p->lm_mode == 1 || p->lm_mode == 2) {                         /* one landmark set: pooled keys (default) or pooled queries */
    pool_single(p, p->lm_mode == 1 ? K : Q, x->L, wf);
    /* The gradient of the kernel holds sign(token - landmark), which is discontinuous: a pooled
       landmark that lies within rounding distance of a token decides that sign differently in
       different precisions.  With lm_f32 the landmark is DEFINED as the single-precision value
       nearest to the exact mean, the precision the device keeps landmarks in, so that both sides
       take the decision on the same numbers. */
    if (p->lm_f32)
      for (size_t e = 0; e < (size_t)m * d; ++e) x->L[e] = (double)(float)x->L[e];
  } else if (p->lm_mode == 3) {                                     /* Alg. 1 as printed: sample query and key landmarks */
    pool_single(p, K, x->L, NULL);
    pool_single(p, Q, x->Lq_own, NULL);
    x->Lq = x->Lq_own;
    if (p->lm_f32)
      for (size_t e = 0; e < (size_t)m * d; ++e) { x->L[e] = (double)(float)x->L[e]; x->Lq[e] = (double)(float)x->Lq[e]; }
  } else memcpy(x->L, Lin, sizeof(double) * (size_t)m * d);
  /* x->L are the key-side landmarks (the only set unless lm_mode 3), x->Lq the query-side ones (the same array otherwise) */
  l1_block(n, m, d, Q, x->L, p->lambda, x->C);                      /* Eq. 8: C = k(Q, K~) */
  l1_block(m, m, d, x->Lq, x->L, p->lambda, x->W);                  /* Eq. 9: W = k(Q~, K~) (ridge added inside Newton-Schulz) */
  l1_block(m, n, d, x->Lq, K, p->lambda, x->R);                     /* k(Q~, K) */
  matmul(m, n, d, x->R, V, x->M);                                   /* M = R V */
  if (p->solver == 1) {                                             /* Sec. 5.3: Y from conjugate gradients on Wr Y = M */
    memset(x->X, 0, sizeof(double) * (size_t)m * m);                /* no inverse is formed */
    cg_solve(m, d, x->W, p->ridge_eps, p->ns_iters, x->M, x->Y);
  } else {
    ns_single(m, x->W, p->ns_iters, p->ridge_eps, p->ns_alpha, x->X, NULL);   /* Alg. 2 */
    matmul(m, m, d, x->X, x->M, x->Y);                              /* Y = X M */
  }
  for (int i = 0; i < n; ++i) {
    if (p->map_mode == 1) {                                         /* Prop. 3 steps 2-4 */
      double mu = 0.0;
      for (int l = 0; l < m; ++l) mu += x->C[(size_t)i * m + l];
      mu /= m;
      for (int l = 0; l < m; ++l)
        x->Z[(size_t)i * m + l] = (s ? s[l] : 1.0) * (x->C[(size_t)i * m + l] - mu) + 1.0 / m;
    } else {
      for (int l = 0; l < m; ++l) x->Z[(size_t)i * m + l] = x->C[(size_t)i * m + l];
    }
  }
  matmul(n, m, d, x->Z, x->Y, O);                                   /* O = Z Y */
}

/*
 * Outputs O [B,H,n,d].  The optional pointers (any may be NULL) receive the
 * intermediates of every head for the pin tests: L [BH,m,d], C [BH,n,m],
 * R [BH,m,n], W [BH,m,m] (before the ridge), X [BH,m,m], M, Y [BH,m,d], Z [BH,n,m].
 * whiten: [H,m] or NULL.
 */
void oracle_fwd(const oracle_problem* p, const double* Q, const double* K, const double* V, const double* Lin,
                const double* whiten, double* O,
                double* oL, double* oC, double* oR, double* oW, double* oX, double* oM, double* oY, double* oZ) {
  int BH = p->B * p->H, n = p->n, d = p->d, m = p->m;
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < BH; ++h) {
    head_ctx x; ctx_alloc(&x, n, d, m);
    size_t nd = (size_t)n * d, md = (size_t)m * d, nm = (size_t)n * m, mm = (size_t)m * m;
    fwd_single(p, Q + h * nd, K + h * nd, V + h * nd, Lin ? Lin + h * md : NULL,
               whiten ? whiten + (size_t)(h % p->H) * m : NULL, head_filter(p, h), &x, O + h * nd);
    if (oL) memcpy(oL + h * md, x.L, sizeof(double) * md);
    if (oC) memcpy(oC + h * nm, x.C, sizeof(double) * nm);
    if (oR) memcpy(oR + h * nm, x.R, sizeof(double) * nm);
    if (oW) memcpy(oW + h * mm, x.W, sizeof(double) * mm);
    if (oX) memcpy(oX + h * mm, x.X, sizeof(double) * mm);
    if (oM) memcpy(oM + h * md, x.M, sizeof(double) * md);
    if (oY) memcpy(oY + h * md, x.Y, sizeof(double) * md);
    if (oZ) memcpy(oZ + h * nm, x.Z, sizeof(double) * nm);
    ctx_free(&x);
  }
}

/*
 * Reverse mode of fwd_single, step by step in reverse order.
 * dL: gradient w.r.t. caller-given landmarks (lm_mode 0) or NULL (lm_mode 1:
 * it is folded into dK through the pooling adjoint).
 */
static void bwd_single(const oracle_problem* p, const double* Q, const double* K, const double* V,
                       const double* Lin, const double* s, const double* wf, const double* dO,
                       double* dQ, double* dK, double* dV, double* dL, double* dwf) {
  /* wf / dwf: this head's landmark-selection filter and its gradient ([taps][d], overwritten), or NULL */
  int n = p->n, d = p->d, m = p->m;
  size_t nd = (size_t)n * d, md = (size_t)m * d, nm = (size_t)n * m, mm = (size_t)m * m;
  head_ctx x; ctx_alloc(&x, n, d, m);
  double* O = (double*)malloc(sizeof(double) * nd);
  fwd_single(p, Q, K, V, Lin, s, wf, &x, O);

  double* dZ = (double*)malloc(sizeof(double) * nm);
  double* dC = (double*)malloc(sizeof(double) * nm);
  double* dY = (double*)malloc(sizeof(double) * md);
  double* dX = (double*)malloc(sizeof(double) * mm);
  double* dM = (double*)malloc(sizeof(double) * md);
  double* dR = (double*)malloc(sizeof(double) * nm);
  double* dW = (double*)malloc(sizeof(double) * mm);
  double* dLt = (double*)calloc(md, sizeof(double));

  matmul_nt(n, d, m, dO, x.Y, dZ);          /* O = Z Y:  dZ = dO Y^T */
  matmul_tn(n, m, d, x.Z, dO, dY);          /*           dY = Z^T dO */
  for (int i = 0; i < n; ++i) {             /* Z_il = s_l (C_il - mean_l' C_il') + 1/m */
    if (p->map_mode == 1) {
      double t = 0.0;
      for (int l = 0; l < m; ++l) t += (s ? s[l] : 1.0) * dZ[(size_t)i * m + l];
      t /= m;
      for (int l = 0; l < m; ++l) dC[(size_t)i * m + l] = (s ? s[l] : 1.0) * dZ[(size_t)i * m + l] - t;
    } else {
      for (int l = 0; l < m; ++l) dC[(size_t)i * m + l] = dZ[(size_t)i * m + l];
    }
  }
  if (p->solver == 1) {
    /* Y solves Wr Y = M (to the accuracy T steps give).  The solve is differentiated as the linear system it
       approximates, each adjoint system by the same T-step method (the paper does not say how its CG kernel is
       differentiated; this is the usual rule for a linear solve):
           dM = Wr^-T dY  ->  CG on Wr dM = dY (Wr is symmetric),      dWr = -dM Y^T. */
    cg_solve(m, d, x.W, p->ridge_eps, p->ns_iters, dY, dM);
    matmul_nt(m, d, m, dM, x.Y, dW);
    for (size_t e = 0; e < mm; ++e) dW[e] = -dW[e];
  } else {
    matmul_nt(m, d, m, dY, x.M, dX);        /* Y = X M:  dX = dY M^T */
    matmul_tn(m, m, d, x.X, dY, dM);        /*           dM = X^T dY */
    ns_single_bwd(m, x.W, p->ns_iters, p->ridge_eps, p->ns_alpha, dX, dW);
  }
  matmul_nt(m, d, n, dM, V, dR);            /* M = R V:  dR = dM V^T */
  matmul_tn(m, n, d, x.R, dM, dV);          /*           dV = R^T dM */

  memset(dQ, 0, sizeof(double) * nd);
  memset(dK, 0, sizeof(double) * nd);
  /* dLt: gradient of the key-side landmarks; dLqt: of the query-side ones (the same accumulator unless lm_mode 3) */
  double* dLq_own = (double*)calloc(md, sizeof(double));
  double* dLqt = (p->lm_mode == 3) ? dLq_own : dLt;
  l1_block_bwd(n, m, d, Q, x.L, p->lambda, x.C, dC, dQ, dLt);      /* C = k(Q, K~) */
  l1_block_bwd(m, n, d, x.Lq, K, p->lambda, x.R, dR, dLqt, dK);    /* R = k(Q~, K) */
  l1_block_bwd(m, m, d, x.Lq, x.L, p->lambda, x.W, dW, dLqt, dLt); /* W = k(Q~, K~) */
  if (dwf) memset(dwf, 0, sizeof(double) * (size_t)((p->gh / p->mh) * (p->gw / p->mw)) * d);
  if (p->lm_mode == 1) pool_single_bwd(p, dLt, dK, K, wf, dwf);
  else if (p->lm_mode == 2) pool_single_bwd(p, dLt, dQ, Q, wf, dwf);
  else if (p->lm_mode == 3) { pool_single_bwd(p, dLt, dK, NULL, NULL, NULL); pool_single_bwd(p, dLqt, dQ, NULL, NULL, NULL); }
  else memcpy(dL, dLt, sizeof(double) * md);
  free(dLq_own);

  free(O); free(dZ); free(dC); free(dY); free(dX); free(dM); free(dR); free(dW); free(dLt);
  ctx_free(&x);
}

void oracle_bwd(const oracle_problem* p, const double* Q, const double* K, const double* V, const double* Lin,
                const double* whiten, const double* dO, double* dQ, double* dK, double* dV, double* dL, double* dfilter) {
  /* dfilter: NULL, or [B*H][taps][d]: the gradient of the landmark-selection filter from each batch element and head
     (the caller adds up the batch elements of a head) */
  int BH = p->B * p->H, n = p->n, d = p->d, m = p->m;
  size_t td = p->lm_filter ? (size_t)((p->gh / p->mh) * (p->gw / p->mw)) * d : 0;
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < BH; ++h) {
    size_t nd = (size_t)n * d, md = (size_t)m * d;
    bwd_single(p, Q + h * nd, K + h * nd, V + h * nd, Lin ? Lin + h * md : NULL,
               whiten ? whiten + (size_t)(h % p->H) * m : NULL, head_filter(p, h), dO + h * nd,
               dQ + h * nd, dK + h * nd, dV + h * nd, dL ? dL + h * md : NULL,
               (dfilter && p->lm_filter) ? dfilter + h * td : NULL);
  }
}

/* ========================================================================= */
/* The steps either side of the path inside the attention block              */
/*   Attention(Q, K, V) = Z V + DWC(V)              (Eq. 7)                   */
/*   rotary position embedding on Q and K           (Sec. 5.1, implementation) */
/* ========================================================================= */

/*
 * Rotary position embedding (Sec. 5.1 adopts RoPE; the rotation is that of the RoFormer paper it cites):
 * token at position p, channel pair (2i, 2i+1), angle theta = p * base^(-2i/d):
 *     x'_{2i} = x_{2i} cos(theta) - x_{2i+1} sin(theta),   x'_{2i+1} = x_{2i} sin(theta) + x_{2i+1} cos(theta).
 * Reading: positions run over the flattened token grid (row-major), p = token index - prefix; the `prefix`
 * leading tokens (class tokens) are not rotated.  inverse != 0 applies the transpose (the adjoint of the map).
 * X, out: [BH, n, d], d even.
 */
void oracle_rope(int BH, int n, int d, int prefix, double base, int inverse, const double* X, double* out) {
#pragma omp parallel for schedule(static)
  for (int bh = 0; bh < BH; ++bh)
    for (int t = 0; t < n; ++t) {
      const double* x = X + ((size_t)bh * n + t) * d;
      double* o = out + ((size_t)bh * n + t) * d;
      for (int i = 0; i < d / 2; ++i) {
        double a = x[2 * i], b = x[2 * i + 1];
        if (t < prefix) { o[2 * i] = a; o[2 * i + 1] = b; continue; }
        double theta = (double)(t - prefix) * pow(base, -2.0 * (double)i / (double)d);
        double c = cos(theta), s = sin(theta);
        if (inverse) s = -s;
        o[2 * i] = a * c - b * s;
        o[2 * i + 1] = a * s + b * c;
      }
    }
}

/*
 * Depth-wise convolution over the value sequence (Eq. 7): every channel c of head h has its own ks x ks filter
 * Wd[h][c][a][b] (ks odd), applied over the gh x gw token grid with zero padding (a cross-correlation, as in every
 * deep-learning framework):
 *     out[r, q, c] = sum_{a, b} Wd[h][c][a][b] * V[r + a - ks/2, q + b - ks/2, c].
 * Reading: the `prefix` leading tokens are not on the grid and receive 0.
 * V, out: [B, H, n, d] with n = prefix + gh * gw; Wd: [H, d, ks, ks].
 */
void oracle_dwc(int B, int H, int n, int d, int prefix, int gh, int gw, int ks, const double* V, const double* Wd, double* out) {
  int half = ks / 2;
#pragma omp parallel for schedule(static)
  for (int bh = 0; bh < B * H; ++bh) {
    int h = bh % H;
    const double* Vh = V + (size_t)bh * n * d;
    double* Oh = out + (size_t)bh * n * d;
    for (int t = 0; t < prefix; ++t)
      for (int c = 0; c < d; ++c) Oh[(size_t)t * d + c] = 0.0;
    for (int r = 0; r < gh; ++r)
      for (int q = 0; q < gw; ++q)
        for (int c = 0; c < d; ++c) {
          double acc = 0.0;
          for (int a = 0; a < ks; ++a)
            for (int b = 0; b < ks; ++b) {
              int rr = r + a - half, qq = q + b - half;
              if (rr < 0 || rr >= gh || qq < 0 || qq >= gw) continue;
              acc += Wd[(((size_t)h * d + c) * ks + a) * ks + b] * Vh[(size_t)(prefix + rr * gw + qq) * d + c];
            }
          Oh[(size_t)(prefix + r * gw + q) * d + c] = acc;
        }
  }
}

/* Adjoint of oracle_dwc: dV [B,H,n,d] and dWd [H,d,ks,ks] (summed over the batch) from dO = dLoss/d out. */
void oracle_dwc_bwd(int B, int H, int n, int d, int prefix, int gh, int gw, int ks, const double* V, const double* Wd,
                    const double* dO, double* dV, double* dWd) {
  int half = ks / 2;
  memset(dV, 0, sizeof(double) * (size_t)B * H * n * d);
  memset(dWd, 0, sizeof(double) * (size_t)H * d * ks * ks);
  for (int bh = 0; bh < B * H; ++bh) {               /* serial over heads: dWd is shared by the batch elements of a head */
    int h = bh % H;
    const double* Vh = V + (size_t)bh * n * d;
    const double* Gh = dO + (size_t)bh * n * d;
    double* dVh = dV + (size_t)bh * n * d;
    for (int r = 0; r < gh; ++r)
      for (int q = 0; q < gw; ++q)
        for (int c = 0; c < d; ++c) {
          double g = Gh[(size_t)(prefix + r * gw + q) * d + c];
          for (int a = 0; a < ks; ++a)
            for (int b = 0; b < ks; ++b) {
              int rr = r + a - half, qq = q + b - half;
              if (rr < 0 || rr >= gh || qq < 0 || qq >= gw) continue;
              size_t wi = (((size_t)h * d + c) * ks + a) * ks + b, vi = (size_t)(prefix + rr * gw + qq) * d + c;
              dVh[vi] += Wd[wi] * g;
              dWd[wi] += Vh[vi] * g;
            }
        }
  }
}
