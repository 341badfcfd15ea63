// C ABI of the Laplacian-Nystrom library: host-side validation, buffer layout and launches.
#include <math.h>
#include <stdlib.h>
#include <stdint.h>
#include <string.h>

#include "../../include/laplace_nystrom.h"
#include "ln_kernels.cuh"
#include "ln_sign2.cuh"
#include "ln_sign3.cuh"
#include "ln_block.cuh"
#include "ln_exact.cuh"
#include <atomic>
#include <mutex>
#include <unordered_map>
#include <type_traits>

using namespace ln;

namespace {

// Number of SMs of the current device (asked once per device; 148 on a B200, the fallback if the query fails).
constexpr int kMaxDevices = 64;
int sm_count() {
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  int v = cached[dev].load(std::memory_order_relaxed);
  if (v <= 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) { cudaGetLastError(); v = 148; }
    cached[dev].store(v, std::memory_order_relaxed);
  }
  return v;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device (again only when a larger size is
// asked for): a table keyed by the kernel's address.
template <typename K>
void want_smem(K kern, size_t smem) {
  static std::mutex mu;
  static std::unordered_map<const void*, int> have[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  const void* id = reinterpret_cast<const void*>(kern);
  std::lock_guard<std::mutex> lk(mu);
  auto it = have[dev].find(id);
  if (it != have[dev].end() && it->second >= (int)smem) return;
  cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  have[dev][id] = (int)smem;
}

template <typename A0, typename... R> A0 arg0(void (*)(A0, R...));   // first parameter type of a kernel (declaration only)
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Bump allocator over a caller-provided buffer; with base == nullptr it only measures.
struct Carver {
  char* base; size_t off;
  explicit Carver(void* b) : base(static_cast<char*>(b)), off(0) {}
  float* take(size_t nfloats) {
    float* p = base ? reinterpret_cast<float*>(base + off) : nullptr;
    off += align_up(nfloats * sizeof(float), 256);
    return p;
  }
};

// Tile of the l1 kernel for a problem: LG landmark groups of QN (4 or 2) landmarks, TG token groups of 8,
// LG * TG <= 256 threads, chosen so that the tiles hug the problem.  Small heads (few pairs per CTA) take
// the two-landmark thread tile, which fits three CTAs per SM.
struct L1Launch { dim3 grid, block; size_t smem; int qn; };
L1Launch plan_l1(int na_max, int nb, int d, int batch, int nprob) {
  const int qn = ((long long)na_max * nb * d <= (1ll << 20)) ? 2 : 4;
  const int lg_cap = (qn == 4) ? 16 : 32;
  int LG = (nb + qn - 1) / qn; if (LG > lg_cap) LG = lg_cap; if (LG < 1) LG = 1;
  int tg_cap = 256 / LG; if (tg_cap > 32) tg_cap = 32;       // at most 256 tokens per tile
  const int groups = (na_max + 7) / 8;
  const int tiles = (groups + tg_cap - 1) / tg_cap;
  int TG = (groups + tiles - 1) / tiles; if (TG < 1) TG = 1;
  L1Launch l;
  l.qn = qn;
  l.block = dim3(LG, TG);
  l.grid = dim3((na_max + 8 * TG - 1) / (8 * TG), batch, nprob);
  l.smem = sizeof(float) * ((size_t)(8 * TG + qn * LG) * L1_PITCH + (size_t)8 * TG * LG);
  return l;
}

std::atomic<bool> g_sign3{true};      // test switch: false = the separate upstream kernels and the two-output sign pass

struct Plan {
  int BH, n, d, m, T, ldm, rpc, chunks;
  size_t scr;                        // floats per scratch matrix of the per-head kernels
  long long hslot;                   // floats per slot of the Newton-Schulz histories
  int s2_tg, s2_rpc, s2_chunks;      // fused sign pass: token groups per tile, tokens per chunk, chunks (0 = not used)
  int s2q_rpc, s2q_chunks;           // the same for the query-side pass, which shares the GPU with the per-head kernel
  int mid_sms;                       // SMs the per-head kernels occupy (Newton-Schulz and its adjoint)
  size_t s2_smem;
  int s3_tiles;                      // sign pass with the upstream factor formed in the kernel: token tiles per head (0 = not used)
  int H, wmode, l1_tiles;            // heads; whitening mode; token tiles of the l1 launch that forms C (statistics partials)
  bool two;                          // two landmark sets (Alg. 1 as printed): W = k(pool(Q), pool(K)) is not symmetric
  bool cg;                           // conjugate gradients in place of Newton-Schulz (fp32 per-head kernels)
};

bool make_plan(const ln_problem* p, Plan* pl) {
  if (!p) return false;
  const int kSMs = sm_count();
  pl->BH = p->B * p->H; pl->n = p->n; pl->d = p->d; pl->m = p->m; pl->T = p->ns_iters;
  pl->ldm = (p->m + 3) & ~3;
  pl->scr = (size_t)p->m * pl->ldm;
  pl->two = p->lm_mode == 3;
  pl->cg = p->solver == 1;
  // the tcgen05 per-head kernels use the symmetry of the landmark kernel matrix; two landmark sets take the general engine
  const bool tcmid = p->dtype == LN_BF16 && !pl->two;
  if (tcmid && p->m > 128) pl->scr = (size_t)kU2Slot;
  // history slots: fp32 [m][ldm], except on the m <= 64 tensor-core path, whose slots hold operand images
  pl->hslot = (long long)p->m * pl->ldm;
  if (tcmid && p->m <= 64) pl->hslot = (long long)(kUmmaMatBytes64 / 4);                 // 16 KiB images >= m * ldm * 4
  if (tcmid && p->m > 64 && p->m <= 128) pl->hslot = (long long)(kUmmaMatBytes / 4);     // 64 KiB images >= m * ldm * 4
  if (tcmid && p->m > 128) pl->hslot = kU2Slot;                                          // four 64 KiB block images
  // token chunks per head for the reductions over tokens: about eight waves of CTAs (two per SM) so that
  // the last wave costs little, but at least 64 tokens per chunk
  const int mblk = (p->m + 63) / 64;
  int want = (16 * kSMs + pl->BH * mblk - 1) / (pl->BH * mblk);
  if (want > 32) want = 32;        // the per-head kernels add up the partial results (eight loads in flight per thread)
  if (want < 1) want = 1;
  int rpc = (p->n + want - 1) / want;
  if (rpc < 256) rpc = 256;
  rpc = (rpc + 31) / 32 * 32;
  pl->rpc = rpc;
  pl->chunks = (p->n + rpc - 1) / rpc;
  // fused sign pass (64-dim slabs): token tiles of 8 * TG tokens that hug n, chunks for about three waves
  pl->s2_tg = pl->s2_rpc = pl->s2_chunks = pl->s2q_rpc = pl->s2q_chunks = 0; pl->s2_smem = 0;
  // per-head kernels (bf16 storage): three CTAs per SM for m <= 64, one for m <= 128, else a cluster of two CTAs per head, one per SM
  pl->mid_sms = p->m <= 64 ? (pl->BH + 2) / 3 : (p->m <= 128 ? pl->BH : kU2Cluster * pl->BH);
  if (p->d % 64 == 0) {
    const int groups = (p->n + 7) / 8;
    int tiles = (groups + S2_TGMAX - 1) / S2_TGMAX;
    int TG = (groups + tiles - 1) / tiles; TG += TG & 1; if (TG > S2_TGMAX) TG = S2_TGMAX; if (TG < 8) TG = 8;
    tiles = (p->n + 8 * TG - 1) / (8 * TG);
    const int slabs = p->d / 64;
    // tiles per chunk: the choice that minimises waves x (time of a CTA), with a CTA's time counted in rounds of 8
    // landmarks plus about three rounds of fixed cost, two CTAs per SM, at most 64 chunks
    const int nrounds = (p->m + S2_RL - 1) / S2_RL;
    auto tiles_per_chunk = [&](int slots) {
      int tpc = tiles; long long best = -1;
      for (int t = 1; t <= tiles; ++t) {
        const int chunks = (tiles + t - 1) / t;
        if (chunks > 64) continue;
        const long long ctas = (long long)pl->BH * slabs * chunks;
        const long long cost = ((ctas + slots - 1) / slots) * ((long long)t * nrounds + 3);
        if (best < 0 || cost < best) { best = cost; tpc = t; }
      }
      return tpc;
    };
    const int tpc = tiles_per_chunk(2 * kSMs);
    pl->s2_tg = TG; pl->s2_rpc = tpc * 8 * TG; pl->s2_chunks = (p->n + pl->s2_rpc - 1) / pl->s2_rpc;
    // The query-side pass runs beside the Newton-Schulz adjoint (one CTA per head on the library's second stream).
    // While that kernel lives, every SM that holds one of its CTAs has one place less for a CTA of the sign pass (both
    // places for 64 < m <= 128, whose CTA fills an SM).  With few heads the pass is planned for the places that are
    // left; with many heads the two kernels take turns anyway and the plan is that of the pass running alone.
    int lost = p->m <= 64 ? pl->BH : (p->m <= 128 ? 2 * pl->BH : 4 * pl->BH);
    if (p->dtype != LN_BF16 || lost > kSMs) lost = 0;
    const int tpq = tiles_per_chunk(2 * kSMs - lost);
    pl->s2q_rpc = tpq * 8 * TG; pl->s2q_chunks = (p->n + pl->s2q_rpc - 1) / pl->s2q_rpc;
    pl->s2_smem = sign2_smem_bytes(p->m);
    if (pl->two) pl->s2_chunks = pl->s2q_chunks = 0;      // two landmark sets: the tcgen05 sign pass or the two plain passes
  }
  // bf16 storage, 64 or 128 dims: one CTA per tile of 8 * TG tokens, upstream factor on the tensor cores in the kernel
  pl->H = p->H; pl->wmode = p->whiten_mode;
  pl->l1_tiles = (int)plan_l1(p->n, p->m, p->d, pl->BH, 1).grid.x;
  pl->s3_tiles = (p->dtype == LN_BF16 && (p->d == 64 || p->d == 128) && g_sign3.load(std::memory_order_relaxed))
                     ? (p->n + 8 * pl->s2_tg - 1) / (8 * pl->s2_tg) : 0;
  return true;
}

// floats of the split operand images of one [m][d] matrix per head (the tcgen05 product kernels read them)
size_t image_floats(const Plan& pl) { return (size_t)((pl.m + GU_KB - 1) / GU_KB) * gu_block_floats(pl.d); }

// Forward context (saved for the backward pass, or carved from ws for inference)
struct Ctx { float *Lf, *C, *Rt, *mu, *W, *Xh, *Ph, *M, *Yt, *ybar, *Yimg, *Y, *cbar, *Lq; NsHdr* hdr; size_t bytes; };
Ctx carve_ctx(const Plan& pl, void* base) {
  Carver c(base); Ctx x;
  const size_t BH = pl.BH, n = pl.n, d = pl.d, m = pl.m;
  x.Lf = c.take(BH * m * d);
  x.C = c.take(BH * n * pl.ldm);
  x.Rt = c.take(BH * n * pl.ldm);
  x.mu = c.take(BH * n);
  x.W = c.take(BH * m * m);
  x.Xh = c.take(BH * (pl.T + 1) * (size_t)pl.hslot);
  x.Ph = c.take(BH * (pl.T > 0 ? pl.T : 1) * (size_t)pl.hslot);   // W X_k (or 2I - W X_k) of the forward pass (tensor-core paths)
  x.M = c.take(BH * m * d);
  x.Yt = c.take(BH * m * d);
  x.ybar = c.take(BH * d);
  x.Yimg = c.take(BH * image_floats(pl));        // Ytilde once more, as split operand images
  x.hdr = reinterpret_cast<NsHdr*>(c.take(BH * (sizeof(NsHdr) / sizeof(float))));
  x.Y = c.take(BH * m * d);                      // Y = X M before the map is folded in (batch-statistic whitening needs it)
  x.cbar = c.take((size_t)pl.H * m);             // column means of C over the batch (batch-statistic whitening)
  x.Lq = c.take(pl.two ? BH * m * d : 0);        // second landmark set (pooled queries); Lf then holds the pooled keys
  x.bytes = c.off;
  return x;
}

struct FwdWs { float *Mpart, *Wr, *P, *cg; double* stat; size_t bytes; };
FwdWs carve_fwd_ws(const Plan& pl, void* base) {
  Carver c(base); FwdWs w;
  const size_t BH = pl.BH, d = pl.d, m = pl.m;
  w.Mpart = c.take(BH * pl.chunks * m * d);
  w.Wr = c.take(BH * pl.scr);
  w.P = c.take(BH * pl.scr);
  w.stat = reinterpret_cast<double*>(c.take(pl.wmode == 1 ? BH * (size_t)pl.l1_tiles * m * 4 : 0));   // [BH][tiles][m][2] doubles
  w.cg = c.take(pl.cg ? BH * 8 * m * d : 0);                    // conjugate gradients: iterate, residual, direction, W times direction (doubles)
  w.bytes = c.off;
  return w;
}

struct BwdWs {
  float *G, *G2, *dYtpart, *dybpart, *dLCpart, *dLRpart, *dY, *dM, *Wr, *P, *Hm, *Ga, *Gb, *dW, *dX, *GW, *dLW, *dLtot, *dKpart, *dMimg, *SB, *kap, *SBq, *dQpart, *dLqtot, *dLW2, *cg;
  size_t bytes;
};
BwdWs carve_bwd_ws(const Plan& pl, void* base) {
  Carver c(base); BwdWs w;
  const size_t BH = pl.BH, n = pl.n, d = pl.d, m = pl.m, ch = pl.chunks;
  size_t chs = pl.s2_chunks > 0 ? (size_t)pl.s2_chunks : ch;     // chunks of the landmark-gradient partials
  size_t chq = pl.s2_chunks > 0 ? (size_t)pl.s2q_chunks : ch;
  if (pl.s3_tiles > 0) chs = chq = (size_t)pl.s3_tiles;
  // upstream factors g of the two token-sized blocks; not materialised when the sign pass forms them itself
  w.G = c.take(pl.s3_tiles > 0 ? 0 : BH * n * pl.ldm);
  w.G2 = c.take(pl.s3_tiles > 0 ? 0 : BH * n * pl.ldm);       // its own buffer: it is formed while the query side reads G
  w.dYtpart = c.take(BH * ch * m * d);
  w.dybpart = c.take(BH * ch * d);
  w.dLCpart = c.take(BH * chq * m * d);
  w.dLRpart = c.take(BH * chs * m * d);
  w.dY = c.take(BH * m * d);
  w.dM = c.take(BH * m * d);
  w.Wr = c.take(BH * pl.scr);
  w.P = c.take(BH * pl.scr);
  w.Hm = c.take(BH * pl.scr);
  w.Ga = c.take(BH * pl.scr);
  w.Gb = c.take(BH * pl.scr);
  w.dW = c.take(BH * pl.scr);
  w.dX = c.take(BH * pl.scr);
  w.GW = c.take(BH * m * pl.ldm);
  w.dLW = c.take(BH * m * d);
  w.dLtot = c.take(BH * m * d);
  w.dKpart = c.take(BH * n * d);
  w.dMimg = c.take(BH * image_floats(pl));
  w.SB = c.take(pl.s3_tiles > 0 ? BH * m * 2 * d : 0);      // scale and offset of every landmark value (folded step)
  w.kap = c.take(pl.wmode == 1 ? (size_t)pl.H * m * 2 : 0); // batch-statistic whitening: (kappa_l, cbar_l) per head and landmark
  // two landmark sets: folded step of the second set, fp32 query gradient before the pooling adjoint, gradient of the
  // second set, column part of the landmark-block sign pass
  w.SBq = c.take(pl.two && pl.s3_tiles > 0 ? BH * m * 2 * d : 0);
  w.dQpart = c.take(pl.two ? BH * n * d : 0);
  w.dLqtot = c.take(pl.two ? BH * m * d : 0);
  w.dLW2 = c.take(pl.two ? BH * m * d : 0);
  w.cg = c.take(pl.cg ? BH * 8 * m * d : 0);
  w.bytes = c.off;
  return w;
}

int validate(const ln_problem* p) {
  if (!p) return LN_ERR_ARG;
  if (p->B <= 0 || p->H <= 0 || p->n <= 0 || p->d <= 0 || p->m <= 0) return LN_ERR_ARG;
  if (p->m > p->n) return LN_ERR_ARG;
  if (!(p->lambda > 0.f) || !isfinite(p->lambda)) return LN_ERR_ARG;
  if (p->ns_iters < 0) return LN_ERR_ARG;
  if (!(p->ridge_eps >= 0.f) || !isfinite(p->ridge_eps)) return LN_ERR_ARG;
  if (!isfinite(p->ns_alpha)) return LN_ERR_ARG;
  if (p->dtype != LN_F32 && p->dtype != LN_BF16) return LN_ERR_ARG;
  if (p->map_mode != 0 && p->map_mode != 1) return LN_ERR_ARG;
  if (p->lm_mode < 0 || p->lm_mode > 3) return LN_ERR_ARG;
  if (p->solver != 0 && p->solver != 1) return LN_ERR_ARG;
  if (p->solver == 1 && (p->lm_mode == 3 || p->whiten_mode == 1)) return LN_ERR_UNSUPPORTED;
  if (p->whiten && !aligned16(p->whiten)) return LN_ERR_ARG;
  if (p->whiten_mode != 0 && p->whiten_mode != 1) return LN_ERR_ARG;
  if (p->whiten_mode == 1) {
    if (p->map_mode != 1 || p->whiten || !p->whiten_batch || !aligned16(p->whiten_batch)) return LN_ERR_ARG;
    if (!(p->whiten_eps >= 0.f) || !isfinite(p->whiten_eps)) return LN_ERR_ARG;
    if (p->lm_mode == 3) return LN_ERR_UNSUPPORTED;
  }
  if (p->lm_mode >= 1) {
    if (p->prefix < 0 || p->gh <= 0 || p->gw <= 0 || p->mh <= 0 || p->mw <= 0) return LN_ERR_ARG;
    if ((long long)p->prefix + (long long)p->gh * p->gw != p->n) return LN_ERR_ARG;
    if ((long long)p->mh * p->mw != p->m) return LN_ERR_ARG;
    if (p->mh > p->gh || p->mw > p->gw) return LN_ERR_ARG;
    if ((long long)p->gh * (p->mh + 1) >= (1ll << 31) || (long long)p->gw * (p->mw + 1) >= (1ll << 31)) return LN_ERR_UNSUPPORTED;
    if ((long long)p->n * p->d / 4 >= (1ll << 32)) return LN_ERR_UNSUPPORTED;
  }
  if (p->lm_filter) {          // depth-wise-convolution landmark selection: r x r regions with stride r, one pooled tensor
    if (p->lm_mode == 0 || !aligned16(p->lm_filter)) return LN_ERR_ARG;
    if (p->gh % p->mh != 0 || p->gw % p->mw != 0) return LN_ERR_ARG;
    if (p->lm_mode == 3) return LN_ERR_UNSUPPORTED;
  }
  if ((long long)p->B * p->H > 65535) return LN_ERR_UNSUPPORTED;
  if (p->d != 32 && p->d != 64 && p->d != 128) return LN_ERR_UNSUPPORTED;
  if (p->m > 256) return LN_ERR_UNSUPPORTED;
  return LN_OK;
}

PoolGeom geom_of(const ln_problem* p) {
  PoolGeom g; g.n = p->n; g.d = p->d; g.m = p->m; g.prefix = p->prefix; g.gh = p->gh; g.gw = p->gw; g.mh = p->mh; g.mw = p->mw;
  g.filt = p->lm_filter; g.H = p->H;
  return g;
}

// A launch that fails is noticed right after it (a later successful call may otherwise hide it) and reported by the
// entry point when it returns.
thread_local bool g_launch_failed = false;
std::atomic<unsigned long long> g_launch_count{0};      // kernels launched by this library since it was loaded
inline void note_launch() {
  g_launch_count.fetch_add(1, std::memory_order_relaxed);
  if (cudaPeekAtLastError() != cudaSuccess) g_launch_failed = true;
}
inline int launch_ok() {
  const bool bad = (cudaGetLastError() != cudaSuccess) || g_launch_failed;
  g_launch_failed = false;
  return bad ? LN_ERR_CUDA : LN_OK;
}
inline unsigned cdiv(long long a, long long b) { return (unsigned)((a + b - 1) / b); }

// Profiling aid: when switched on by ln_trace_begin every launch is bracketed by two CUDA events
// on its stream.  Off by default; the product path never touches it.
constexpr int kTraceCap = 2048;
struct Trace {
  std::atomic<bool> on{false};
  int count = 0;
  cudaEvent_t ev[2 * kTraceCap];
  const char* name[kTraceCap];
} g_trace;
struct TraceScope {
  cudaStream_t st; int slot;
  TraceScope(const char* name, cudaStream_t s) : st(s), slot(-1) {
    if (g_trace.on && g_trace.count < kTraceCap) {
      slot = g_trace.count++;
      g_trace.name[slot] = name;
      cudaEventRecord(g_trace.ev[2 * slot], st);
    }
  }
  ~TraceScope() { if (slot >= 0) cudaEventRecord(g_trace.ev[2 * slot + 1], st); }
};
#define LN_LAUNCH(name, st, ...) do { TraceScope ts_(name, st); __VA_ARGS__; note_launch(); } while (0)

// Side stream.  The per-head kernels (Newton-Schulz and its adjoint: one CTA or cluster per head, bound by the
// latency of a chain of small products) do not depend on the token-sized kernels next to them, so the entry
// points enqueue them on a second stream of the library, forked from and joined back into the caller's stream
// with events: to the caller everything is still ordered on the stream it passed.  Switched off while a trace is
// recorded (so that the per-launch times are those of kernels running alone) and by ln_set_overlap(0).
// One side stream and a ring of events per (device, caller stream), kept in a small table: calls on different
// streams (or from different host threads on different streams) share nothing, so they neither serialise on a
// common side stream nor wait on one another's events.  Two host threads that enqueue on the SAME stream at the same
// time are not supported (the order of their work on that stream would be undefined anyway).
constexpr int kSideSlots = 32, kSideEvents = 16;
struct SideState { bool used = false, ok = false; int dev = -1; cudaStream_t caller = nullptr; cudaStream_t s = nullptr;
                   cudaEvent_t ev[kSideEvents]; unsigned next = 0; bool side_tried = false;
                   // copy streams of the host-buffer entry point (created on its first call for this caller stream)
                   bool copy_tried = false, copy_ok = false; cudaStream_t cin = nullptr, cout = nullptr; cudaEvent_t cev[6]; };
SideState g_side[kSideSlots];
std::mutex g_side_mu;
std::atomic<bool> g_overlap{true};
struct Side {
  cudaStream_t s = nullptr; cudaEvent_t fork_ev[2] = {nullptr, nullptr}, join_ev = nullptr;
  bool on() const { return s != nullptr; }
  // everything enqueued on `st` so far precedes what is enqueued on the side stream from now on (k-th fork of a call)
  void fork(cudaStream_t st, int k = 0) const { cudaEventRecord(fork_ev[k], st); cudaStreamWaitEvent(s, fork_ev[k], 0); }
  // everything enqueued on the side stream so far precedes what is enqueued on `st` from now on
  void join(cudaStream_t st) const { cudaEventRecord(join_ev, s); cudaStreamWaitEvent(st, join_ev, 0); }
  // a join in two halves (uses the second fork event): mark() notes what the side stream holds so far, join_mark()
  // makes `st` wait for exactly that, whatever was enqueued on the side stream in between
  void mark() const { cudaEventRecord(fork_ev[1], s); }
  void join_mark(cudaStream_t st) const { cudaStreamWaitEvent(st, fork_ev[1], 0); }
};
Side side_acquire(bool want, cudaStream_t caller) {
  Side r;
  if (!want || !g_overlap.load(std::memory_order_relaxed) || g_trace.on.load(std::memory_order_relaxed)) return r;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return r;
  std::lock_guard<std::mutex> lk(g_side_mu);
  SideState* d = nullptr;
  for (int i = 0; i < kSideSlots && !d; ++i)
    if (g_side[i].used && g_side[i].dev == dev && g_side[i].caller == caller) d = &g_side[i];
  if (!d) {
    for (int i = 0; i < kSideSlots && !d; ++i) if (!g_side[i].used) d = &g_side[i];
    if (!d) return r;                  // table full: this caller stream runs without overlap
    d->used = true; d->dev = dev; d->caller = caller;
  }
  if (!d->side_tried) {
    d->side_tried = true;
    // highest priority: its few large CTAs (up to a whole SM each) are placed before the pending small CTAs of
    // the kernels on the caller's stream, which would otherwise keep every SM partly occupied until their grids end
    int prio_lo = 0, prio_hi = 0;
    bool ok = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess;
    ok = ok && cudaStreamCreateWithPriority(&d->s, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
    for (int i = 0; ok && i < kSideEvents; ++i) ok = cudaEventCreateWithFlags(&d->ev[i], cudaEventDisableTiming) == cudaSuccess;
    d->ok = ok;
    if (!ok) cudaGetLastError();
  }
  if (!d->ok) return r;
  r.s = d->s; r.fork_ev[0] = d->ev[d->next]; r.fork_ev[1] = d->ev[d->next + 1]; r.join_ev = d->ev[d->next + 2];
  d->next = (d->next + 4) % kSideEvents;
  return r;
}

// Two copy streams per (device, caller stream) for the host-buffer entry point: host -> device copies on one, device ->
// host copies on the other, tied to the caller's stream by events, so that a step's copies run beside its own kernels
// (the copy of O back beside the backward pass, the copy of dO in beside the forward pass) and PCIe carries both
// directions at once.  To the caller everything is still ordered on the stream it passed.  ok == false (creation
// failed, or no room in the table): the entry point puts everything on the caller's stream.
struct CopyStreams { bool ok = false; cudaStream_t cin = nullptr, cout = nullptr; cudaEvent_t ev[6] = {}; };
CopyStreams copy_acquire(cudaStream_t caller) {
  CopyStreams r;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return r;
  std::lock_guard<std::mutex> lk(g_side_mu);
  SideState* d = nullptr;
  for (int i = 0; i < kSideSlots && !d; ++i)
    if (g_side[i].used && g_side[i].dev == dev && g_side[i].caller == caller) d = &g_side[i];
  if (!d) {
    for (int i = 0; i < kSideSlots && !d; ++i) if (!g_side[i].used) d = &g_side[i];
    if (!d) return r;
    d->used = true; d->dev = dev; d->caller = caller;      // the compute side stream of this slot is created by side_acquire when first asked for
  }
  if (!d->copy_tried) {
    d->copy_tried = true;
    bool ok = cudaStreamCreateWithFlags(&d->cin, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&d->cout, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 6; ++i) ok = cudaEventCreateWithFlags(&d->cev[i], cudaEventDisableTiming) == cudaSuccess;
    d->copy_ok = ok;
    if (!ok) cudaGetLastError();
  }
  if (!d->copy_ok) return r;
  r.ok = true; r.cin = d->cin; r.cout = d->cout;
  for (int i = 0; i < 6; ++i) r.ev[i] = d->cev[i];
  return r;
}

// Launch with `cl` CTAs per thread-block cluster (cl = 1: an ordinary launch).
constexpr int kMidCluster = 4;     // CTAs that share one head on the general (two landmark sets) engine beyond 64 landmarks
template <typename... KArgs, typename... Args>
void launch_clustered(void (*kern)(KArgs...), int grid, int cl, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cl; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// landmark pooling: one thread per (landmark, 4 channels) for small bins, a CTA per landmark for large ones
template <typename T>
void launch_pool(const ln_problem* p, const T* src, float* L, cudaStream_t st) {
  const int bin_tokens = ((p->gh + p->mh - 1) / p->mh) * ((p->gw + p->mw - 1) / p->mw);
  if (bin_tokens >= 64) LN_LAUNCH("k_pool", st, k_pool_wide<T><<<dim3(p->m, p->B * p->H), 256, 0, st>>>(src, L, geom_of(p)));
  else LN_LAUNCH("k_pool", st, k_pool<T><<<dim3(cdiv(p->m, 256 / (p->d / 4)), p->B * p->H), 256, 0, st>>>(src, L, geom_of(p)));
}

template <typename T> constexpr int is_f32() { return std::is_same<T, float>::value ? 1 : 0; }

L1Prob l1_prob(const void* A, int a_f32, float* E, float* rowsum, int na, int d, int lde, float rs_scale, double* stat = nullptr) {
  L1Prob q; q.A = A; q.E = E; q.rowsum = rowsum; q.sA = (long long)na * d; q.sE = (long long)na * lde;
  q.na = na; q.lde = lde; q.a_f32 = a_f32; q.rs_scale = rs_scale; q.stat = stat;
  return q;
}

void launch_l1_args(const char* name, L1Args& a, int nprob, int batch, cudaStream_t st) {
  int na_max = 0;
  for (int i = 0; i < nprob; ++i) na_max = a.p[i].na > na_max ? a.p[i].na : na_max;
  L1Launch l = plan_l1(na_max, a.nb, a.d, batch, nprob);
  // a single block without row sums (the stand-alone entry point on few, large matrices): the landmark range is split
  // over blockIdx.z until the launch has about two CTAs per SM
  a.jsplits = 1;
  if (nprob == 1 && !a.p[0].rowsum && !a.p[0].stat) {
    const long long ctas = (long long)l.grid.x * l.grid.y, tb = (long long)l.qn * l.block.x;
    long long sp = (2ll * sm_count() + ctas - 1) / ctas;
    const long long tiles = (a.nb + tb - 1) / tb;
    if (sp > tiles) sp = tiles;
    if (sp > 1) { a.jsplits = (int)sp; l.grid.z = (unsigned)sp; }
  }
  if (l.qn == 4) {
    want_smem(k_l1<4>, l.smem);
    LN_LAUNCH(name, st, k_l1<4><<<l.grid, l.block, l.smem, st>>>(a));
  } else {
    want_smem(k_l1<2>, l.smem);
    LN_LAUNCH(name, st, k_l1<2><<<l.grid, l.block, l.smem, st>>>(a));
  }
}

template <typename TA, typename TB>
void launch_l1(const char* name, const TA* A, const TB* Bm, float* E, float* rowsum, int batch, int na, int nb, int d,
               int lde, float lambda, cudaStream_t st, float rs_scale = 1.f) {
  L1Args a;
  a.p[0] = l1_prob(A, is_f32<TA>(), E, rowsum, na, d, lde, rs_scale);
  a.p[1] = a.p[0]; a.p[2] = a.p[0];
  a.Bm = Bm; a.sB = (long long)nb * d; a.nb = nb; a.d = d; a.b_f32 = is_f32<TB>();
  a.nscale = -1.4426950408889634f / lambda;
  launch_l1_args(name, a, 1, batch, st);
}

// ------------------------------------------------------------------------------------------
template <typename T, int D>
int fwd_impl(const ln_problem* p, const Plan& pl, const T* Q, const T* K, const T* V, const T* L, T* O,
             const Ctx& x, const FwdWs& w, int32_t* dev_status, cudaStream_t st, bool clear_status, const DwcEpi* epi = nullptr) {
  // epi: NULL, or the convolution branch DWC(V) of the attention block, added in the epilogue of the O product (bf16, d = 64 / 128)
  const int BH = pl.BH, n = pl.n, m = pl.m, kSMs = sm_count();
  if (dev_status && clear_status) cudaMemsetAsync(dev_status, 0, sizeof(int32_t) * BH, st);   // the kernels OR their flags into it
  // landmarks (Sec. 4.2)
  const bool two = pl.two;    // two landmark sets: Lf = pooled keys (columns of C and W), Lq = pooled queries (rows of W, columns of R^T)
  if (two) {
    launch_pool<T>(p, K, x.Lf, st);
    launch_pool<T>(p, Q, x.Lq, st);
  } else if (p->lm_mode >= 1) {      // pooled keys, or pooled queries (lm_mode 2)
    launch_pool<T>(p, p->lm_mode == 1 ? K : Q, x.Lf, st);
  } else {
    const long long cnt = (long long)BH * m * D;
    LN_LAUNCH("k_to_f32", st, k_to_f32<T><<<cdiv(cnt, 256), 256, 0, st>>>(L, x.Lf, cnt));
  }
  // the three kernel blocks: C = k(Q,L) with its row sums, R^T = k(K,L), W = k(L,L)
  // (not for many small heads, where the per-head kernel fills the GPU and the split launches cost more than the
  // overlap returns)
  const Side side = side_acquire(!two && !pl.cg && std::is_same<T, bf16>::value && (2 * pl.mid_sms <= kSMs || (long long)n * m * D > (1ll << 22)), st);
  const bool umma_prod = std::is_same<T, bf16>::value && (D == 64 || D == 128);   // tcgen05 products over the landmarks
  // Where the iteration is expected to outlast the two token-sized blocks (few heads of few tokens), only the iteration
  // goes to the side stream; estimates in microseconds: 5 / 12 / 100 per step for m <= 64 / <= 128 / larger, and the l1
  // blocks at about half of the FP32 peak
  const double ns_us = pl.T * (m <= 64 ? 5.0 : (m <= 128 ? 12.0 : 100.0));
  const double l1_us = 2.0 * 2.0 * n * m * D * BH / 20e6;
  const bool bw = p->whiten_mode == 1;              // batch-statistic whitening: s comes out of the kernel block C of this call
  const float* const whiten_eff = bw ? p->whiten_batch : p->whiten;
  const bool deep = side.on() && l1_us >= ns_us && !bw;   // (the map fold then has to wait for C: no work is left to run beside it)
  const float* const Mparts_src = w.Mpart;
  const int Mparts = pl.chunks == 1 ? 0 : pl.chunks;
  // Newton-Schulz (phase bit 0) and Y = X M with the folded map (phase bit 1), one CTA or cluster per head
  auto launch_mid = [&](cudaStream_t s, int phase) {
    constexpr bool TC = std::is_same<T, bf16>::value;
    auto launch = [&](auto kern, size_t smem, int cl = 1) {
      want_smem(kern, smem);
      LN_LAUNCH(phase == 3 ? "k_mid_fwd" : (phase == 1 ? "k_mid_fwd_ns" : "k_mid_fwd_y"), s,
                launch_clustered(kern, BH * cl, cl, smem, s, m, pl.ldm, pl.T, p->ridge_eps, p->ns_alpha, p->H, p->map_mode,
                                 whiten_eff, x.W, w.Wr, w.P, x.Xh, x.Ph, x.hdr, Mparts_src, Mparts, x.M, x.Y, x.Yt,
                                 x.ybar, dev_status, pl.hslot, umma_prod ? reinterpret_cast<bf16*>(x.Yimg) : nullptr, phase,
                                 pl.cg ? 1 : 0, w.cg));
    };
    // conjugate gradients (Sec. 5.3): fp32, one CTA per head, whatever the storage type
    if (pl.cg) { launch(k_mid_fwd<D, false, 0>, sizeof(NsSmem)); return; }
    // general (non-symmetric) matrix: the mma.sync or FFMA engine, shared by the CTAs of a cluster beyond 64 landmarks
    if (two && m > 64) launch(k_mid_fwd<D, TC, 0, kMidCluster>, sizeof(NsSmem), kMidCluster);
    else if (two) launch(k_mid_fwd<D, TC, 0>, sizeof(NsSmem));
    else if (TC && m <= 64) launch(k_mid_fwd<D, TC, TC ? 64 : 0>, 3 * kUmmaMatBytes64);
    else if (TC && m <= 128) launch(k_mid_fwd<D, TC, TC ? 128 : 0>, 3 * kUmmaMatBytes);
    else if (TC) launch(k_mid_fwd<D, TC, TC ? 256 : 0, TC ? kU2Cluster : 1>, 3 * kUmmaMatBytes, kU2Cluster);   // m > 128: a cluster per head
    else launch(k_mid_fwd<D, TC, 0>, sizeof(NsSmem));
  };
  {
    L1Args a;
    a.Bm = x.Lf; a.sB = (long long)m * D; a.nb = m; a.d = D; a.b_f32 = 1;
    a.nscale = -1.4426950408889634f / p->lambda;
    const L1Prob pc = l1_prob(Q, is_f32<T>(), x.C, p->map_mode == 1 ? x.mu : nullptr, n, D, pl.ldm, 1.f / (float)m,  // row means (Prop. 3 step 2)
                              bw ? w.stat : nullptr);                                                                    // column statistics (Eq. 5)
    const L1Prob pr = l1_prob(K, is_f32<T>(), x.Rt, nullptr, n, D, pl.ldm, 1.f);
    const L1Prob pw = l1_prob(two ? x.Lq : x.Lf, 1, x.W, nullptr, m, D, m, 1.f);
    if (two) {
      // C = k(Q, pool K) and W = k(pool Q, pool K) share their landmark operand; R^T = k(K, pool Q) has its own
      a.p[0] = pc; a.p[1] = pw; a.p[2] = pw;
      launch_l1_args("l1_CW", a, 2, BH, st);
      a.Bm = x.Lq;
      a.p[0] = pr; a.p[1] = pr; a.p[2] = pr;
      launch_l1_args("l1_R", a, 1, BH, st);
    } else if (side.on()) {
      // W first: the iteration on it runs beside the token-sized blocks.  Then R^T: M = R V (bound by memory) and the
      // rest of the per-head work run beside the query block C (bound by arithmetic), which only the last product needs.
      a.p[0] = pw; a.p[1] = pw; a.p[2] = pw;
      launch_l1_args("l1_W", a, 1, BH, st);
      side.fork(st, 0);
      launch_mid(side.s, 1);
      if (deep) {
        a.p[0] = pr; a.p[1] = pr; a.p[2] = pr;
        launch_l1_args("l1_R", a, 1, BH, st);
        side.fork(st, 1);
      } else {
        a.p[0] = pc; a.p[1] = pr; a.p[2] = pr;
        launch_l1_args("l1_CR", a, 2, BH, st);
      }
    } else {
      a.p[0] = pc; a.p[1] = pr; a.p[2] = pw;
      launch_l1_args("l1_CRW", a, 3, BH, st);
    }
  }
  // M = R V, partial over token chunks (a single chunk writes M itself)
  float* const Mdst = pl.chunks == 1 ? x.M : w.Mpart;
  const cudaStream_t sm_ = deep ? side.s : st;               // stream of M = R V and of what follows from it
  if constexpr (std::is_same<T, bf16>::value)
  {
    want_smem(k_tn_mma<D>, tn_mma_smem<D>());
    LN_LAUNCH("tn_M", sm_, k_tn_mma<D><<<dim3(pl.chunks, cdiv(m, 64), BH), 256, tn_mma_smem<D>(), sm_>>>(x.Rt, pl.ldm, nullptr, V, Mdst, nullptr, n, m, pl.rpc));
  }
  else
    LN_LAUNCH("tn_M", sm_, k_tn<T, D><<<dim3(pl.chunks, cdiv(m, 64), BH), 256, 0, sm_>>>(x.Rt, pl.ldm, nullptr, V, Mdst, nullptr, n, m, pl.rpc));
  // whitening scale from the statistics the C block left (Eq. 6), before the map is folded
  if (bw) LN_LAUNCH("k_wstat_final", st, k_wstat_final<<<dim3(cdiv(m, 32), p->H), 256, 0, st>>>(w.stat, p->B, p->H, n, m, pl.l1_tiles, p->whiten_eps,
                                                                                               p->whiten_batch, x.cbar));
  // Newton-Schulz, Y = X M, folded map
  if (side.on() && !deep) { side.join(st); launch_mid(st, 2); }
  else if (side.on()) {
    launch_mid(side.s, 2);
    L1Args a;
    a.Bm = x.Lf; a.sB = (long long)m * D; a.nb = m; a.d = D; a.b_f32 = 1;
    a.nscale = -1.4426950408889634f / p->lambda;
    a.p[0] = l1_prob(Q, is_f32<T>(), x.C, p->map_mode == 1 ? x.mu : nullptr, n, D, pl.ldm, 1.f / (float)m);
    a.p[1] = a.p[0]; a.p[2] = a.p[0];
    launch_l1_args("l1_C", a, 1, BH, st);
    side.join(st);
  } else launch_mid(st, 3);
  // O = (C - mu) Ytilde + ybar
  if constexpr (std::is_same<T, bf16>::value && (D == 64 || D == 128)) {
    if (epi && epi->src) {
      const size_t smem = nn_umma_stage_dwc<D>() + (size_t)epi->ks * epi->ks * D * sizeof(float);
      want_smem(k_nn_umma<D, true>, smem);
      LN_LAUNCH("nn_O", st, k_nn_umma<D, true><<<dim3(cdiv(n, 128), BH), 256, smem, st>>>(x.C, pl.ldm, p->map_mode == 1 ? x.mu : nullptr,
                                                                                      reinterpret_cast<const bf16*>(x.Yimg), x.ybar, O, n, m, dev_status, *epi));
    } else {
      const size_t smem = nn_umma_smem<D>();
      want_smem(k_nn_umma<D>, smem);
      LN_LAUNCH("nn_O", st, k_nn_umma<D><<<dim3(cdiv(n, 128), BH), 256, smem, st>>>(x.C, pl.ldm, p->map_mode == 1 ? x.mu : nullptr,
                                                                                reinterpret_cast<const bf16*>(x.Yimg), x.ybar, O, n, m, dev_status, DwcEpi()));
    }
  } else if constexpr (std::is_same<T, bf16>::value)
    LN_LAUNCH("nn_O", st, k_nn_mma<D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(x.C, pl.ldm, p->map_mode == 1 ? x.mu : nullptr, x.Yt, x.ybar, O, n, m));
  else
    LN_LAUNCH("nn_O", st, k_nn<T, D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(x.C, pl.ldm, p->map_mode == 1 ? x.mu : nullptr, x.Yt, x.ybar, O, n, m));
  return launch_ok();
}

template <typename T, int D>
int bwd_impl(const ln_problem* p, const Plan& pl, const T* Q, const T* K, const T* V, const T* dO,
             const Ctx& x, const BwdWs& w, T* dQ, T* dK, T* dV, T* dL, int32_t* dev_status, cudaStream_t st, bool clear_status,
             const DwcEpi* epi = nullptr) {
  // epi: NULL, or the adjoint DWC^T(dO) of the block's convolution branch, added in the epilogue of the dV product
  const int BH = pl.BH, n = pl.n, m = pl.m, ch = pl.chunks, kSMs = sm_count();
  const float inv_lambda = 1.f / p->lambda;
  const float* mu = p->map_mode == 1 ? x.mu : nullptr;
  if (dev_status && clear_status) cudaMemsetAsync(dev_status, 0, sizeof(int32_t) * BH, st);
  // query side: Z'^T dO and column sums of dO; g^C = (dO Ytilde^T) o C / lambda; dQ; landmark part
  auto launch_tn_dY = [&](cudaStream_t s) {
    if constexpr (std::is_same<T, bf16>::value)
    {
      want_smem(k_tn_mma<D>, tn_mma_smem<D>());
      LN_LAUNCH("tn_dY", s, k_tn_mma<D><<<dim3(ch, cdiv(m, 64), BH), 256, tn_mma_smem<D>(), s>>>(x.C, pl.ldm, mu, dO, w.dYtpart, w.dybpart, n, m, pl.rpc));
    }
    else
      LN_LAUNCH("tn_dY", s, k_tn<T, D><<<dim3(ch, cdiv(m, 64), BH), 256, 0, s>>>(x.C, pl.ldm, mu, dO, w.dYtpart, w.dybpart, n, m, pl.rpc));
  };
  auto launch_ntg_C = [&]() {
    if constexpr (std::is_same<T, bf16>::value) {
      if constexpr (D == 64 || D == 128) {
        want_smem(k_ntg_umma<D>, ntg_umma_smem<D>());
        LN_LAUNCH("ntg_C", st, k_ntg_umma<D><<<dim3(cdiv(n, 128), BH), 256, ntg_umma_smem<D>(), st>>>(dO, reinterpret_cast<const bf16*>(x.Yimg), x.C, pl.ldm,
                                                                                                  w.G, n, m, inv_lambda, dev_status));
      } else
        LN_LAUNCH("ntg_C", st, k_nt_g_mma<D><<<dim3(cdiv(n, 64), cdiv(m, 64), BH), 256, 0, st>>>(dO, x.Yt, x.C, pl.ldm, w.G, n, m, inv_lambda));
    } else {
      LN_LAUNCH("ntg_C", st, k_nt_g<T, D><<<dim3(cdiv(n, 64), cdiv(m, 64), BH), 256, 0, st>>>(dO, x.Yt, x.C, pl.ldm, w.G, n, m, inv_lambda));
    }
  };
  const bool fused_sign = pl.s2_chunks > 0;
  const bool poolQ = p->lm_mode == 2;                 // the token-side gradient that still needs the pooling adjoint is dQ, not dK
  const bool two = pl.two;                            // two landmark sets: both token-side gradients need a pooling adjoint
  const float* const LfC = x.Lf;                      // landmarks of the query-side block C (pooled keys when two)
  const float* const LfR = two ? x.Lq : x.Lf;         // landmarks of the key-side block R^T (pooled queries when two)
  // fp32 row outputs of the sign passes that a pooling adjoint still follows (NULL: the pass writes the gradient itself)
  float* const qrows_f = two ? w.dQpart : (poolQ ? w.dKpart : nullptr);
  float* const krows_f = (two || !poolQ) ? w.dKpart : nullptr;
  const bool sign3 = pl.s3_tiles > 0;                 // the sign passes form their upstream factor themselves (tcgen05)
  const int chs = sign3 ? pl.s3_tiles : (fused_sign ? pl.s2_chunks : ch);
  const int chq = sign3 ? pl.s3_tiles : (fused_sign ? pl.s2q_chunks : ch);    // chunks of the query-side landmark-gradient partials
  // one sign pass of a token-sized block: tokens, upstream operands (U, pre-split images of Y), kernel block A
  const bool bw = p->whiten_mode == 1;                // batch-statistic whitening: the scale is the forward pass's own estimate
  const float* const whiten_eff = bw ? p->whiten_batch : p->whiten;
  auto launch_sign3 = [&](const char* name, const T* tokp, const T* Up, const float* Yimgp, const float* Ap, auto* rowsp, float* partp,
                          const float* SBp, const float* kap = nullptr) {
    if constexpr (std::is_same<T, bf16>::value && (D == 64 || D == 128)) {
      auto go = [&](auto kern) {
        want_smem(kern, sign3_smem_bytes());
        LN_LAUNCH(name, st, kern<<<dim3(pl.s3_tiles, D / 64, BH), dim3(16, pl.s2_tg), sign3_smem_bytes(), st>>>(
                      tokp, SBp, Up, reinterpret_cast<const bf16*>(Yimgp), Ap, pl.ldm, rowsp, partp, n, m, inv_lambda, dev_status, kap, p->H));
      };
      using TO = std::remove_pointer_t<decltype(rowsp)>;
      if (pl.s2_tg == S3_TGMAX) go(k_sign3<TO, D, 1, true>); else go(k_sign3<TO, D, 2, true>);
    }
  };
  // The per-head kernel and the landmark-block sign pass need Z'^T dO only: with a side stream they run beside
  // the query-side kernels and are joined before the key side, which needs dM.
  const Side side = side_acquire(std::is_same<T, bf16>::value, st);
  const bool umma_prod = std::is_same<T, bf16>::value && (D == 64 || D == 128);
  auto launch_mid = [&](cudaStream_t s, int phase = 3) {
    constexpr bool TC = std::is_same<T, bf16>::value;
    auto launch = [&](auto kern, size_t smem, int cl = 1) {
      want_smem(kern, smem);
      LN_LAUNCH(phase == 3 ? "k_mid_bwd" : (phase == 1 ? "k_mid_bwd_dM" : "k_mid_bwd_adj"), s,
                launch_clustered(kern, BH * cl, cl, smem, s, m, pl.T, p->H, p->map_mode, inv_lambda, pl.ldm, whiten_eff,
                                                 x.W, x.Xh, x.Ph, x.hdr, x.M, w.dYtpart, w.dybpart, ch, p->ridge_eps, w.Wr, w.P,
                                                 w.Hm, w.Ga, w.Gb, w.dW, w.dX, w.dY, w.dM, w.GW, dev_status, pl.hslot,
                                                 umma_prod ? reinterpret_cast<bf16*>(w.dMimg) : nullptr, two ? 0 : 1,
                                                 pl.cg ? 1 : 0, x.Y, w.cg, phase));
    };
    if (pl.cg) { launch(k_mid_bwd<D, false, 0>, sizeof(NsSmem)); return; }
    if (two && m > 64) launch(k_mid_bwd<D, TC, 0, kMidCluster>, sizeof(NsSmem), kMidCluster);
    else if (two) launch(k_mid_bwd<D, TC, 0>, sizeof(NsSmem));
    else if (TC && m <= 64) launch(k_mid_bwd<D, TC, TC ? 64 : 0>, 4 * kUmmaMatBytes64);
    else if (TC && m <= 128) launch(k_mid_bwd<D, TC, TC ? 128 : 0>, 3 * kUmmaMatBytes);
    else if (TC) launch(k_mid_bwd<D, TC, TC ? 256 : 0, TC ? kU2Cluster : 1>, 3 * kUmmaMatBytes, kU2Cluster);
    else launch(k_mid_bwd<D, TC, 0>, sizeof(NsSmem));
  };
  // key-side products: g^R = (V dM^T) o R^T / lambda and dV = R^T dM (they need dM from the per-head kernel)
  auto launch_ntg_R = [&](cudaStream_t s) {
    if constexpr (std::is_same<T, bf16>::value) {
      if constexpr (D == 64 || D == 128) {
        want_smem(k_ntg_umma<D>, ntg_umma_smem<D>());
        LN_LAUNCH("ntg_R", s, k_ntg_umma<D><<<dim3(cdiv(n, 128), BH), 256, ntg_umma_smem<D>(), s>>>(V, reinterpret_cast<const bf16*>(w.dMimg), x.Rt, pl.ldm,
                                                                                                w.G2, n, m, inv_lambda, dev_status));
      } else
        LN_LAUNCH("ntg_R", s, k_nt_g_mma<D><<<dim3(cdiv(n, 64), cdiv(m, 64), BH), 256, 0, s>>>(V, w.dM, x.Rt, pl.ldm, w.G2, n, m, inv_lambda));
    } else {
      LN_LAUNCH("ntg_R", s, k_nt_g<T, D><<<dim3(cdiv(n, 64), cdiv(m, 64), BH), 256, 0, s>>>(V, w.dM, x.Rt, pl.ldm, w.G2, n, m, inv_lambda));
    }
  };
  auto launch_nn_dV = [&](cudaStream_t s) {
    if constexpr (std::is_same<T, bf16>::value) {
      if constexpr (D == 64 || D == 128) {
        if (epi && epi->src) {
          const size_t smem = nn_umma_stage_dwc<D>() + (size_t)epi->ks * epi->ks * D * sizeof(float);
          want_smem(k_nn_umma<D, true>, smem);
          LN_LAUNCH("nn_dV", s, k_nn_umma<D, true><<<dim3(cdiv(n, 128), BH), 256, smem, s>>>(x.Rt, pl.ldm, nullptr, reinterpret_cast<const bf16*>(w.dMimg),
                                                                                         nullptr, dV, n, m, dev_status, *epi));
        } else {
          const size_t smem = nn_umma_smem<D>();
          want_smem(k_nn_umma<D>, smem);
          LN_LAUNCH("nn_dV", s, k_nn_umma<D><<<dim3(cdiv(n, 128), BH), 256, smem, s>>>(x.Rt, pl.ldm, nullptr, reinterpret_cast<const bf16*>(w.dMimg),
                                                                                   nullptr, dV, n, m, dev_status, DwcEpi()));
        }
      } else
        LN_LAUNCH("nn_dV", s, k_nn_mma<D><<<dim3(cdiv(n, 64), BH), 256, 0, s>>>(x.Rt, pl.ldm, nullptr, w.dM, nullptr, dV, n, m));
    } else {
      LN_LAUNCH("nn_dV", s, k_nn<T, D><<<dim3(cdiv(n, 64), BH), 256, 0, s>>>(x.Rt, pl.ldm, nullptr, w.dM, nullptr, dV, n, m));
    }
  };
  auto launch_sign_W = [&](cudaStream_t s) {
    // one set: GW is symmetrised, so the row pass carries both roles of L.  Two sets: rows -> pooled queries, columns -> pooled keys
    LN_LAUNCH("sign_rows_dLW", s, k_sign_rows<float, float, float, D><<<dim3(cdiv(m, 64), BH), 256, 0, s>>>(LfR, LfC, w.GW, pl.ldm, w.dLW, m, m));
    if (two) LN_LAUNCH("sign_cols_dLW", s, k_sign_cols<float, float, D><<<dim3(1, cdiv(m, 64), BH), 256, 0, s>>>(LfR, LfC, w.GW, pl.ldm, w.dLW2, m, m, (m + 31) / 32 * 32));
  };
  // Side stream: the per-head kernel, the landmark-block sign pass and dV (bound by latency and by memory) run beside
  // the sign passes (bound by arithmetic).  The upstream of the key-side block, which the second sign pass waits for,
  // joins them where the query-side sign pass is long enough to hide it (large heads); for small heads it follows the
  // first sign pass on the caller's stream, so that only the per-head kernel stands between the two sign passes.
  const bool ntg_on_side = side.on() && (long long)n * m * D > (1ll << 22);
  // Z'^T dO is needed by the per-head kernel only: it goes to the side stream too unless that stream is expected to be
  // the longer one anyway (estimates in microseconds: 7 / 16 / 30 per step and wave of heads for m <= 64 / <= 128 /
  // larger; the sign pass at 0.43 of the FP32 peak, 0.25 for small launches)
  const int mid_waves = (int)(m <= 64 ? cdiv(BH, 3 * kSMs) : (m <= 128 ? cdiv(BH, kSMs) : cdiv((long long)kU2Cluster * BH, kSMs)));
  const double side_us = pl.T * (m <= 64 ? 7.0 : (m <= 128 ? 16.0 : 30.0)) * mid_waves;
  const double sign_ops = 3.0 * n * m * D * BH;
  const double main_us = sign_ops / (37.2e6 * (sign_ops > 4e9 ? 0.43 : 0.25));
  const bool tn_on_side = side.on() && side_us < 0.8 * main_us && !bw;
  if (!tn_on_side) launch_tn_dY(st);
  // Batch-statistic whitening: ds needs Z'^T dO of every batch element of a head, and the query-side sign pass needs
  // the coefficient it gives, so Z'^T dO stays on the caller's stream in front of both.
  const float* const kap = bw ? w.kap : nullptr;
  if (bw) LN_LAUNCH("k_whiten_bwd", st, k_whiten_bwd<<<dim3(cdiv(m, 8), p->H), 256, 0, st>>>(x.Y, w.dYtpart, ch, p->whiten_batch, x.cbar, p->B, p->H,
                                                                                            n, m, D, w.kap));
  if (side.on()) {
    side.fork(st);
    if (tn_on_side) launch_tn_dY(side.s);
    // with the sign passes forming their factor themselves, the second one waits for dM only: the per-head kernel runs
    // as two launches and the adjoint of the iteration, which nothing token-sized needs, follows the mark
    const bool split_mid = sign3 && !pl.cg;
    launch_mid(side.s, split_mid ? 1 : 3);
    if (ntg_on_side && !sign3) launch_ntg_R(side.s);
    side.mark();                     // what the second sign pass needs from this stream ends here
    if (split_mid) launch_mid(side.s, 2);
    launch_nn_dV(side.s);
    launch_sign_W(side.s);
  }
  if (sign3) {
    const long long cnt = (long long)BH * m * D;
    LN_LAUNCH("k_fold_landmarks", st, k_fold_landmarks<<<cdiv(cnt, 256), 256, 0, st>>>(LfC, w.SB, D, cnt));
    if (two) LN_LAUNCH("k_fold_landmarks", st, k_fold_landmarks<<<cdiv(cnt, 256), 256, 0, st>>>(LfR, w.SBq, D, cnt));
    if (qrows_f) launch_sign3("sign3_dQ_dLC", Q, dO, x.Yimg, x.C, qrows_f, w.dLCpart, w.SB, kap);
    else launch_sign3("sign3_dQ_dLC", Q, dO, x.Yimg, x.C, dQ, w.dLCpart, w.SB, kap);
  } else {
    launch_ntg_C();
    if (bw) LN_LAUNCH("k_g_whiten_add", st, k_g_whiten_add<<<dim3(cdiv((long long)n * pl.ldm, 256), BH), 256, 0, st>>>(w.G, x.C, w.kap, p->H, n, m, pl.ldm, inv_lambda));
  }
  if (sign3) {
  } else if (fused_sign) {
    auto launch2 = [&](const char* name, auto kern, const T* tokp, auto* rowsp, float* partp) {
      want_smem(kern, pl.s2_smem);
      LN_LAUNCH(name, st, kern<<<dim3(chq, D / 64, BH), dim3(16, pl.s2_tg), pl.s2_smem, st>>>(tokp, x.Lf, w.G, pl.ldm, rowsp, partp, n, m, D, pl.s2q_rpc));
    };
    if (poolQ) {
      if (pl.s2_tg == S2_TGMAX) launch2("sign2_dQ_dLC", k_sign2<T, float, 1>, Q, w.dKpart, w.dLCpart);
      else launch2("sign2_dQ_dLC", k_sign2<T, float, 2>, Q, w.dKpart, w.dLCpart);
    } else {
      if (pl.s2_tg == S2_TGMAX) launch2("sign2_dQ_dLC", k_sign2<T, T, 1>, Q, dQ, w.dLCpart);
      else launch2("sign2_dQ_dLC", k_sign2<T, T, 2>, Q, dQ, w.dLCpart);
    }
  } else {
    if (qrows_f) LN_LAUNCH("sign_rows_dQ", st, k_sign_rows<T, float, float, D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(Q, LfC, w.G, pl.ldm, qrows_f, n, m));
    else LN_LAUNCH("sign_rows_dQ", st, k_sign_rows<T, float, T, D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(Q, LfC, w.G, pl.ldm, dQ, n, m));
    LN_LAUNCH("sign_cols_dLC", st, k_sign_cols<T, float, D><<<dim3(ch, cdiv(m, 64), BH), 256, 0, st>>>(Q, LfC, w.G, pl.ldm, w.dLCpart, n, m, pl.rpc));
  }
  if (side.on()) { side.join_mark(st); if (!ntg_on_side && !sign3) launch_ntg_R(st); }
  else { launch_mid(st); launch_sign_W(st); if (!sign3) launch_ntg_R(st); launch_nn_dV(st); }
  // key side: dK (kernel part); landmark part
  if (sign3) {
    if (!krows_f) launch_sign3("sign3_dK_dLR", K, V, w.dMimg, x.Rt, dK, w.dLRpart, two ? w.SBq : w.SB);
    else launch_sign3("sign3_dK_dLR", K, V, w.dMimg, x.Rt, krows_f, w.dLRpart, two ? w.SBq : w.SB);
  } else if (fused_sign) {
    auto launch2 = [&](const char* name, auto kern, const T* tokp, auto* rowsp, float* partp) {
      want_smem(kern, pl.s2_smem);
      LN_LAUNCH(name, st, kern<<<dim3(chs, D / 64, BH), dim3(16, pl.s2_tg), pl.s2_smem, st>>>(tokp, x.Lf, w.G2, pl.ldm, rowsp, partp, n, m, D, pl.s2_rpc));
    };
    if (poolQ) {
      if (pl.s2_tg == S2_TGMAX) launch2("sign2_dK_dLR", k_sign2<T, T, 1>, K, dK, w.dLRpart);
      else launch2("sign2_dK_dLR", k_sign2<T, T, 2>, K, dK, w.dLRpart);
    } else {
      if (pl.s2_tg == S2_TGMAX) launch2("sign2_dK_dLR", k_sign2<T, float, 1>, K, w.dKpart, w.dLRpart);
      else launch2("sign2_dK_dLR", k_sign2<T, float, 2>, K, w.dKpart, w.dLRpart);
    }
  } else {
    if (!krows_f) LN_LAUNCH("sign_rows_dK", st, k_sign_rows<T, float, T, D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(K, LfR, w.G2, pl.ldm, dK, n, m));
    else LN_LAUNCH("sign_rows_dK", st, k_sign_rows<T, float, float, D><<<dim3(cdiv(n, 64), BH), 256, 0, st>>>(K, LfR, w.G2, pl.ldm, krows_f, n, m));
    LN_LAUNCH("sign_cols_dLR", st, k_sign_cols<T, float, D><<<dim3(ch, cdiv(m, 64), BH), 256, 0, st>>>(K, LfR, w.G2, pl.ldm, w.dLRpart, n, m, pl.rpc));
  }
  // landmark gradient and its way back to the keys
  if (side.on()) side.join(st);      // dV and the landmark-block part are complete
  const int md = m * D;
  if (two) {                  // pooled keys: columns of C and of W; pooled queries: columns of R^T and rows of W
    LN_LAUNCH("k_reduce3", st, k_reduce3_wide<float><<<dim3(cdiv(md, 128), BH), 256, 0, st>>>(w.dLCpart, chq, w.dLW2, 1, nullptr, 0, w.dLtot, md));
    LN_LAUNCH("k_reduce3", st, k_reduce3_wide<float><<<dim3(cdiv(md, 128), BH), 256, 0, st>>>(w.dLRpart, chs, w.dLW, 1, nullptr, 0, w.dLqtot, md));
    LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<T><<<dim3(cdiv((long long)n * (D / 4), 256 * POOL_EPT), BH), 256, 0, st>>>(w.dKpart, w.dLtot, dK, geom_of(p), 1));
    LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<T><<<dim3(cdiv((long long)n * (D / 4), 256 * POOL_EPT), BH), 256, 0, st>>>(w.dQpart, w.dLqtot, dQ, geom_of(p), 1));
  } else if (p->lm_mode >= 1) {      // the landmark gradient returns to the pooled tensor (keys, or queries for lm_mode 2)
    if (chq + chs >= 16) LN_LAUNCH("k_reduce3", st, k_reduce3_wide<float><<<dim3(cdiv(md, 128), BH), 256, 0, st>>>(w.dLCpart, chq, w.dLRpart, chs, w.dLW, 1, w.dLtot, md));
    else LN_LAUNCH("k_reduce3", st, k_reduce3<float><<<dim3(cdiv(md, 1024), BH), 256, 0, st>>>(w.dLCpart, chq, w.dLRpart, chs, w.dLW, 1, w.dLtot, md));
    LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<T><<<dim3(cdiv((long long)n * (D / 4), 256 * POOL_EPT), BH), 256, 0, st>>>(w.dKpart, w.dLtot, poolQ ? dQ : dK, geom_of(p), 1));
    if (p->lm_filter) {          // gradient of the selection filter, summed over the batch elements of a head
      const int taps = (p->gh / p->mh) * (p->gw / p->mw);
      // the (batch element, landmark) pairs are split over enough CTAs to fill the GPU; the partial sums go to the query-side
      // landmark partials of the sign pass, which k_reduce3 has consumed by now
      const long long room = (long long)BH * chq * m * D / ((long long)p->H * taps * D);
      long long splits = cdiv(4ll * kSMs, (long long)taps * p->H);
      if (splits > (long long)p->B * m / 64) splits = (long long)p->B * m / 64;
      if (splits > room) splits = room;
      if (splits > 65535) splits = 65535;
      if (splits < 1) splits = 1;
      float* fpart = splits > 1 ? w.dLCpart : p->lm_filter_grad;
      LN_LAUNCH("k_filter_grad", st, k_filter_grad<T><<<dim3(taps, p->H, (unsigned)splits), 256, 0, st>>>(poolQ ? Q : K, w.dLtot, fpart, geom_of(p), p->B));
      if (splits > 1) {
        const int count = p->H * taps * D;
        LN_LAUNCH("k_filter_reduce", st, k_filter_reduce<<<cdiv(count, 1024), 256, 0, st>>>(w.dLCpart, (int)splits, p->lm_filter_grad, count));
      }
    }
  } else {
    if (chq + chs >= 16) LN_LAUNCH("k_reduce3", st, k_reduce3_wide<T><<<dim3(cdiv(md, 128), BH), 256, 0, st>>>(w.dLCpart, chq, w.dLRpart, chs, w.dLW, 1, dL, md));
    else LN_LAUNCH("k_reduce3", st, k_reduce3<T><<<dim3(cdiv(md, 1024), BH), 256, 0, st>>>(w.dLCpart, chq, w.dLRpart, chs, w.dLW, 1, dL, md));
    LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<T><<<dim3(cdiv((long long)n * (D / 4), 256 * POOL_EPT), BH), 256, 0, st>>>(w.dKpart, nullptr, dK, geom_of(p), 0));
  }
  return launch_ok();
}

template <typename T>
int fwd_dispatch_d(const ln_problem* p, const Plan& pl, const void* Q, const void* K, const void* V, const void* L,
                   void* O, const Ctx& x, const FwdWs& w, int32_t* ds, cudaStream_t st, bool clear_status, const DwcEpi* epi) {
  const T *q = (const T*)Q, *k = (const T*)K, *v = (const T*)V, *l = (const T*)L; T* o = (T*)O;
  switch (p->d) {
    case 32: return fwd_impl<T, 32>(p, pl, q, k, v, l, o, x, w, ds, st, clear_status, epi);
    case 64: return fwd_impl<T, 64>(p, pl, q, k, v, l, o, x, w, ds, st, clear_status, epi);
    case 128: return fwd_impl<T, 128>(p, pl, q, k, v, l, o, x, w, ds, st, clear_status, epi);
  }
  return LN_ERR_UNSUPPORTED;
}
template <typename T>
int bwd_dispatch_d(const ln_problem* p, const Plan& pl, const void* Q, const void* K, const void* V, const void* dO,
                   const Ctx& x, const BwdWs& w, void* dQ, void* dK, void* dV, void* dL, int32_t* ds, cudaStream_t st, bool clear_status,
                   const DwcEpi* epi) {
  const T *q = (const T*)Q, *k = (const T*)K, *v = (const T*)V, *g = (const T*)dO;
  switch (p->d) {
    case 32: return bwd_impl<T, 32>(p, pl, q, k, v, g, x, w, (T*)dQ, (T*)dK, (T*)dV, (T*)dL, ds, st, clear_status, epi);
    case 64: return bwd_impl<T, 64>(p, pl, q, k, v, g, x, w, (T*)dQ, (T*)dK, (T*)dV, (T*)dL, ds, st, clear_status, epi);
    case 128: return bwd_impl<T, 128>(p, pl, q, k, v, g, x, w, (T*)dQ, (T*)dK, (T*)dV, (T*)dL, ds, st, clear_status, epi);
  }
  return LN_ERR_UNSUPPORTED;
}

// ---- stand-alone ns_pinv scratch
struct NsWs { float *Wr, *P, *Hm, *Ga, *Gb, *Xh; NsHdr* hdr; size_t bytes; };
NsWs carve_ns_ws(int batch, int m, int T, void* base) {
  Carver c(base); NsWs w;
  const size_t mm = (size_t)m * m, b = batch;
  w.Wr = c.take(b * mm); w.P = c.take(b * mm); w.Hm = c.take(b * mm); w.Ga = c.take(b * mm); w.Gb = c.take(b * mm);
  w.Xh = c.take(b * (T + 1) * mm);
  w.hdr = reinterpret_cast<NsHdr*>(c.take(b * (sizeof(NsHdr) / sizeof(float))));
  w.bytes = c.off;
  return w;
}

// CTAs of a thread-block cluster that share one matrix of the stand-alone Newton-Schulz entry points (64 x 64 output
// tiles of every product are dealt out to them)
int ns_cluster(int m) { return m > 128 ? 8 : (m > 64 ? 4 : 1); }
void launch_ns_pinv(int batch, int m, int iters, float eps, float alpha, const float* W, const NsWs& w, float* Xh, float* X,
                    float* resid, cudaStream_t st) {
  const int cl = ns_cluster(m);
  auto go = [&](auto kern) {
    LN_LAUNCH("k_ns_pinv", st, launch_clustered(kern, batch * cl, cl, 0, st, m, iters, eps, alpha, W, w.Wr, w.P, Xh, w.hdr, X, resid));
  };
  if (cl == 8) go(k_ns_pinv<8>); else if (cl == 4) go(k_ns_pinv<4>); else go(k_ns_pinv<1>);
}
}  // namespace

namespace {
struct L1BwdWs { float *Kmat, *part, *rowpart; int rpc, chunks, lper, lsplits; size_t bytes; };
L1BwdWs carve_l1bwd(int batch, int na, int nb, int d, void* base) {
  Carver c(base); L1BwdWs w;
  // rows of A per CTA of the pass over the columns: whole 64-column tiles, about two CTAs per SM in all
  const int coltiles = (nb + 63) / 64;
  int want = (2 * sm_count() + batch * coltiles - 1) / (batch * coltiles); if (want < 1) want = 1;
  int rpc = (na + want - 1) / want; rpc = (rpc + 31) / 32 * 32;
  w.rpc = rpc; w.chunks = (na + rpc - 1) / rpc;
  // columns per CTA of the pass over the rows: split while the 64-row tiles alone are fewer than two CTAs per SM
  const int rowtiles = (na + 63) / 64;
  int sp = (2 * sm_count() + batch * rowtiles - 1) / (batch * rowtiles);
  if (sp > (nb + 31) / 32) sp = (nb + 31) / 32;
  if (sp < 1) sp = 1;
  w.lper = ((nb + sp - 1) / sp + 31) / 32 * 32;
  w.lsplits = (nb + w.lper - 1) / w.lper;
  w.Kmat = c.take((size_t)batch * na * nb);
  w.part = c.take((size_t)batch * w.chunks * nb * d);
  w.rowpart = c.take(w.lsplits > 1 ? (size_t)batch * w.lsplits * na * d : 0);
  w.bytes = c.off;
  return w;
}
template <typename T, int D>
void l1_bwd_impl(int batch, int na, int nb, const T* A, const T* Bm, float lambda, const float* Kmat, const float* dK,
                 T* dA, T* dB, const L1BwdWs& w, cudaStream_t st) {
  if (!Kmat) { launch_l1<T, T>("l1_kernel", A, Bm, w.Kmat, nullptr, batch, na, nb, D, nb, lambda, st); Kmat = w.Kmat; }
  // the factor dK o K / lambda is formed where the two passes load their tiles of it
  const float il = 1.f / lambda;
  if (w.lsplits > 1) {
    LN_LAUNCH("k_sign_rows", st, k_sign_rows<T, T, float, D><<<dim3(cdiv(na, 64), batch, w.lsplits), 256, 0, st>>>(A, Bm, dK, nb, w.rowpart, na, nb, w.lper, Kmat, il));
    LN_LAUNCH("k_reduce3", st, k_reduce3<T><<<dim3(cdiv(na * D, 1024), batch), 256, 0, st>>>(w.rowpart, w.lsplits, nullptr, 0, nullptr, 0, dA, na * D));
  } else {
    LN_LAUNCH("k_sign_rows", st, k_sign_rows<T, T, T, D><<<dim3(cdiv(na, 64), batch), 256, 0, st>>>(A, Bm, dK, nb, dA, na, nb, 0, Kmat, il));
  }
  LN_LAUNCH("k_sign_cols", st, k_sign_cols<T, T, D><<<dim3(w.chunks, cdiv(nb, 64), batch), 256, 0, st>>>(A, Bm, dK, nb, w.part, na, nb, w.rpc, Kmat, il));
  LN_LAUNCH("k_reduce3", st, k_reduce3<T><<<dim3(cdiv(nb * D, 1024), batch), 256, 0, st>>>(w.part, w.chunks, nullptr, 0, nullptr, 0, dB, nb * D));
}
}  // namespace

// ==========================================================================================
extern "C" {

int ln_trace_begin(void) {
  if (g_trace.on) return LN_ERR_ARG;
  for (int i = 0; i < 2 * kTraceCap; ++i)
    if (cudaEventCreate(&g_trace.ev[i]) != cudaSuccess) return LN_ERR_CUDA;
  g_trace.count = 0;
  g_trace.on = true;
  return LN_OK;
}

int ln_trace_end(int32_t capacity, int32_t* count, float* ms, const char** names) {
  if (!g_trace.on || !count || capacity < 0) return LN_ERR_ARG;
  g_trace.on = false;
  int status = LN_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) status = LN_ERR_CUDA;
  *count = g_trace.count;
  for (int i = 0; i < g_trace.count && i < capacity && status == LN_OK; ++i) {
    if (ms && cudaEventElapsedTime(&ms[i], g_trace.ev[2 * i], g_trace.ev[2 * i + 1]) != cudaSuccess) status = LN_ERR_CUDA;
    if (names) names[i] = g_trace.name[i];
  }
  for (int i = 0; i < 2 * kTraceCap; ++i) cudaEventDestroy(g_trace.ev[i]);
  return status;
}

uint64_t ln_launch_count(void) { return (uint64_t)g_launch_count.load(std::memory_order_relaxed); }

int ln_set_fused_sign(int enabled) { return g_sign3.exchange(enabled != 0) ? 1 : 0; }

int ln_set_overlap(int enabled) {
  return g_overlap.exchange(enabled != 0) ? 1 : 0;
}

const char* ln_status_string(int s) {
  switch (s) {
    case LN_OK: return "ok";
    case LN_ERR_ARG: return "invalid argument";
    case LN_ERR_UNSUPPORTED: return "outside the supported envelope";
    case LN_ERR_WORKSPACE: return "workspace too small";
    case LN_ERR_CUDA: return "CUDA launch failed";
    case LN_ERR_STATIC_LIMIT: return "problem exceeds the static scratch of the no-allocation entry point";
  }
  return "unknown status";
}

size_t laplace_nystrom_saved_bytes(const ln_problem* p) {
  if (validate(p) != LN_OK) return 0;
  Plan pl; make_plan(p, &pl);
  return carve_ctx(pl, nullptr).bytes;
}

size_t laplace_nystrom_workspace_bytes(const ln_problem* p, int32_t with_saved) {
  if (validate(p) != LN_OK) return 0;
  Plan pl; make_plan(p, &pl);
  const size_t f = carve_fwd_ws(pl, nullptr).bytes, b = carve_bwd_ws(pl, nullptr).bytes;
  size_t ws = f > b ? f : b;
  if (!with_saved) ws = f + carve_ctx(pl, nullptr).bytes;
  return ws;
}

}  // extern "C"

namespace {
// host-side checks of the attention entry points; nothing is enqueued when one fails
int check_fwd_args(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L, const void* O,
                   const void* saved, const void* ws, size_t ws_bytes) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (!Q || !K || !V || !O || !ws) return LN_ERR_ARG;
  if ((p->lm_mode == 0) != (L != nullptr)) return LN_ERR_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) || !aligned16(L) ||
      !aligned16(saved))
    return LN_ERR_ARG;
  if (ws_bytes < laplace_nystrom_workspace_bytes(p, saved != nullptr)) return LN_ERR_WORKSPACE;
  return LN_OK;
}
int check_bwd_args(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L, const void* dO,
                   const void* saved, const void* dQ, const void* dK, const void* dV, const void* dL, const void* ws,
                   size_t ws_bytes) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (!Q || !K || !V || !dO || !saved || !dQ || !dK || !dV || !ws) return LN_ERR_ARG;
  if ((p->lm_mode == 0) != (L != nullptr)) return LN_ERR_ARG;
  if ((p->lm_mode == 0) != (dL != nullptr)) return LN_ERR_ARG;
  if (p->lm_filter && (!p->lm_filter_grad || !aligned16(p->lm_filter_grad))) return LN_ERR_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(saved) || !aligned16(dQ) ||
      !aligned16(dK) || !aligned16(dV) || !aligned16(dL) || !aligned16(ws))
    return LN_ERR_ARG;
  if (ws_bytes < laplace_nystrom_workspace_bytes(p, 1)) return LN_ERR_WORKSPACE;
  return LN_OK;
}
// clear_status: zero dev_status first (the stand-alone entry points); the host-buffer step clears it once and lets
// the backward pass OR its flags into what the forward pass left
int fwd_entry(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L, void* O,
              void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream, bool clear_status, const DwcEpi* epi = nullptr) {
  const int s = check_fwd_args(p, Q, K, V, L, O, saved, ws, ws_bytes);
  if (s != LN_OK) return s;
  Plan pl; make_plan(p, &pl);
  const FwdWs w = carve_fwd_ws(pl, ws);
  const Ctx x = carve_ctx(pl, saved ? saved : static_cast<char*>(ws) + w.bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (p->dtype == LN_F32) return fwd_dispatch_d<float>(p, pl, Q, K, V, L, O, x, w, dev_status, st, clear_status, epi);
  return fwd_dispatch_d<bf16>(p, pl, Q, K, V, L, O, x, w, dev_status, st, clear_status, epi);
}
int bwd_entry(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L,
              const void* dO, const void* saved, void* dQ, void* dK, void* dV, void* dL, void* ws,
              size_t ws_bytes, int32_t* dev_status, void* stream, bool clear_status, const DwcEpi* epi = nullptr) {
  const int s = check_bwd_args(p, Q, K, V, L, dO, saved, dQ, dK, dV, dL, ws, ws_bytes);
  if (s != LN_OK) return s;
  Plan pl; make_plan(p, &pl);
  const BwdWs w = carve_bwd_ws(pl, ws);
  const Ctx x = carve_ctx(pl, const_cast<void*>(saved));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (p->dtype == LN_F32) return bwd_dispatch_d<float>(p, pl, Q, K, V, dO, x, w, dQ, dK, dV, dL, dev_status, st, clear_status, epi);
  return bwd_dispatch_d<bf16>(p, pl, Q, K, V, dO, x, w, dQ, dK, dV, dL, dev_status, st, clear_status, epi);
}
}  // namespace

extern "C" {

int laplace_nystrom_fwd(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L, void* O,
                        void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  return fwd_entry(p, Q, K, V, L, O, saved, ws, ws_bytes, dev_status, stream, true);
}

int laplace_nystrom_bwd(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L,
                        const void* dO, const void* saved, void* dQ, void* dK, void* dV, void* dL, void* ws,
                        size_t ws_bytes, int32_t* dev_status, void* stream) {
  return bwd_entry(p, Q, K, V, L, dO, saved, dQ, dK, dV, dL, ws, ws_bytes, dev_status, stream, true);
}


namespace {
// splits of the token rows per head for the whitening statistics: about eight CTAs per SM, at least 64 rows each
void wstat_plan(const ln_problem* p, int* nsplit, int* rows_per_split) {
  const int BH = p->B * p->H;
  int sp = (8 * sm_count() + BH - 1) / BH;
  if (sp > 64) sp = 64;
  if (sp > (p->n + 63) / 64) sp = (p->n + 63) / 64;
  if (sp < 1) sp = 1;
  int rps = (p->n + sp - 1) / sp;
  rps = (rps + 3) / 4 * 4;
  *rows_per_split = rps;
  *nsplit = (p->n + rps - 1) / rps;
}
}  // namespace

size_t laplace_nystrom_whiten_stats_workspace_bytes(const ln_problem* p) {
  if (validate(p) != LN_OK) return 0;
  int sp, rps; wstat_plan(p, &sp, &rps);
  return align_up((size_t)p->B * p->H * sp * p->m * 2 * sizeof(double), 256);
}

int laplace_nystrom_whiten_stats(const ln_problem* p, const void* saved, float eps_w, float* whiten_out, void* ws,
                                 size_t ws_bytes, void* stream) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (!saved || !whiten_out || !ws) return LN_ERR_ARG;
  if (!(eps_w >= 0.f) || !isfinite(eps_w)) return LN_ERR_ARG;
  if (!aligned16(saved) || !aligned16(whiten_out) || !aligned16(ws)) return LN_ERR_ARG;
  if (ws_bytes < laplace_nystrom_whiten_stats_workspace_bytes(p)) return LN_ERR_WORKSPACE;
  Plan pl; make_plan(p, &pl);
  const Ctx x = carve_ctx(pl, const_cast<void*>(saved));
  int sp, rps; wstat_plan(p, &sp, &rps);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* part = static_cast<double*>(ws);
  LN_LAUNCH("k_wstat_part", st, k_wstat_part<<<dim3(sp, pl.BH), 256, 0, st>>>(x.C, pl.ldm, p->n, p->m, rps, part));
  LN_LAUNCH("k_wstat_final", st, k_wstat_final<<<dim3(cdiv(p->m, 32), p->H), 256, 0, st>>>(part, p->B, p->H, p->n, p->m, sp, eps_w, whiten_out, nullptr));
  return launch_ok();
}

size_t laplace_nystrom_host_staging_bytes(const ln_problem* p) {
  if (validate(p) != LN_OK) return 0;
  const size_t one = ((size_t)p->B * p->H * p->n * p->d * (p->dtype == LN_F32 ? 4 : 2) + 255) / 256 * 256;
  return 8 * one;                                  // Q, K, V, dO in; O, dQ, dK, dV out
}

int laplace_nystrom_fwd_bwd_host(const ln_problem* p, const void* hQ, const void* hK, const void* hV, const void* hdO,
                                 void* hO, void* hdQ, void* hdK, void* hdV, void* staging, size_t staging_bytes,
                                 void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (p->lm_mode < 1) return LN_ERR_UNSUPPORTED;
  if (!hQ || !hK || !hV || !hdO || !hO || !hdQ || !hdK || !hdV || !staging || !saved || !ws) return LN_ERR_ARG;
  if (!aligned16(staging)) return LN_ERR_ARG;
  if (staging_bytes < laplace_nystrom_host_staging_bytes(p)) return LN_ERR_WORKSPACE;
  const size_t bytes = (size_t)p->B * p->H * p->n * p->d * (p->dtype == LN_F32 ? 4 : 2);
  const size_t one = (bytes + 255) / 256 * 256;
  char* d = static_cast<char*>(staging);
  // every check of the two passes comes before the first copy: an argument error enqueues nothing
  s = check_fwd_args(p, d, d + one, d + 2 * one, nullptr, d + 4 * one, saved, ws, ws_bytes);
  if (s != LN_OK) return s;
  s = check_bwd_args(p, d, d + one, d + 2 * one, nullptr, d + 3 * one, saved, d + 5 * one, d + 6 * one, d + 7 * one,
                     nullptr, ws, ws_bytes);
  if (s != LN_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const void* hin[4] = {hQ, hK, hV, hdO};
  void* hout[3] = {hdQ, hdK, hdV};
  const CopyStreams cs = g_overlap.load(std::memory_order_relaxed) ? copy_acquire(st) : CopyStreams();
  if (!cs.ok) {                       // everything on the caller's stream, one after the other
    for (int i = 0; i < 4; ++i)
      if (cudaMemcpyAsync(d + i * one, hin[i], bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return LN_ERR_CUDA;
    s = fwd_entry(p, d, d + one, d + 2 * one, nullptr, d + 4 * one, saved, ws, ws_bytes, dev_status, stream, true);
    if (s != LN_OK) return s;
    if (cudaMemcpyAsync(hO, d + 4 * one, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LN_ERR_CUDA;
    // the backward pass ORs its flags into the status words the forward pass cleared and wrote
    s = bwd_entry(p, d, d + one, d + 2 * one, nullptr, d + 3 * one, saved, d + 5 * one, d + 6 * one, d + 7 * one,
                  nullptr, ws, ws_bytes, dev_status, stream, false);
    if (s != LN_OK) return s;
    for (int i = 0; i < 3; ++i)
      if (cudaMemcpyAsync(hout[i], d + (5 + i) * one, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LN_ERR_CUDA;
    return LN_OK;
  }
  // Copies on the two copy streams: Q, K, V in, then dO in beside the forward pass; O out beside the backward pass; the
  // three gradients out at the end.  ev[0]: what the caller's stream held before this call (it may still use the
  // staging buffers); ev[1]: Q, K, V have arrived; ev[2]: dO has arrived; ev[3]: forward pass done; ev[4]: backward
  // pass done; ev[5]: every copy out done, which the caller's stream waits for before the call counts as complete.
  bool okc = cudaEventRecord(cs.ev[0], st) == cudaSuccess;
  okc = okc && cudaStreamWaitEvent(cs.cin, cs.ev[0], 0) == cudaSuccess && cudaStreamWaitEvent(cs.cout, cs.ev[0], 0) == cudaSuccess;
  for (int i = 0; okc && i < 3; ++i) okc = cudaMemcpyAsync(d + i * one, hin[i], bytes, cudaMemcpyHostToDevice, cs.cin) == cudaSuccess;
  okc = okc && cudaEventRecord(cs.ev[1], cs.cin) == cudaSuccess;
  okc = okc && cudaMemcpyAsync(d + 3 * one, hin[3], bytes, cudaMemcpyHostToDevice, cs.cin) == cudaSuccess;
  okc = okc && cudaEventRecord(cs.ev[2], cs.cin) == cudaSuccess;
  okc = okc && cudaStreamWaitEvent(st, cs.ev[1], 0) == cudaSuccess;
  if (!okc) return LN_ERR_CUDA;
  s = fwd_entry(p, d, d + one, d + 2 * one, nullptr, d + 4 * one, saved, ws, ws_bytes, dev_status, stream, true);
  if (s != LN_OK) return s;
  okc = cudaEventRecord(cs.ev[3], st) == cudaSuccess && cudaStreamWaitEvent(cs.cout, cs.ev[3], 0) == cudaSuccess;
  okc = okc && cudaMemcpyAsync(hO, d + 4 * one, bytes, cudaMemcpyDeviceToHost, cs.cout) == cudaSuccess;
  okc = okc && cudaStreamWaitEvent(st, cs.ev[2], 0) == cudaSuccess;
  if (!okc) return LN_ERR_CUDA;
  // the backward pass ORs its flags into the status words the forward pass cleared and wrote
  s = bwd_entry(p, d, d + one, d + 2 * one, nullptr, d + 3 * one, saved, d + 5 * one, d + 6 * one, d + 7 * one,
                nullptr, ws, ws_bytes, dev_status, stream, false);
  if (s != LN_OK) return s;
  okc = cudaEventRecord(cs.ev[4], st) == cudaSuccess && cudaStreamWaitEvent(cs.cout, cs.ev[4], 0) == cudaSuccess;
  for (int i = 0; okc && i < 3; ++i) okc = cudaMemcpyAsync(hout[i], d + (5 + i) * one, bytes, cudaMemcpyDeviceToHost, cs.cout) == cudaSuccess;
  okc = okc && cudaEventRecord(cs.ev[5], cs.cout) == cudaSuccess && cudaStreamWaitEvent(st, cs.ev[5], 0) == cudaSuccess;
  return okc ? LN_OK : LN_ERR_CUDA;
}

size_t ns_pinv_workspace_bytes(int32_t batch, int32_t m, int32_t iters) {
  if (batch <= 0 || m <= 0 || iters < 0) return 0;
  return carve_ns_ws(batch, m, iters, nullptr).bytes;
}

int ns_pinv(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha, float* X,
            float* X_hist, float* resid, void* ws, size_t ws_bytes, void* stream) {
  if (batch <= 0 || m <= 0 || iters < 0 || !W || !X || !ws) return LN_ERR_ARG;
  if (!(ridge_eps >= 0.f) || !isfinite(ridge_eps) || !isfinite(alpha)) return LN_ERR_ARG;
  if (!aligned16(W) || !aligned16(X) || !aligned16(X_hist) || !aligned16(ws)) return LN_ERR_ARG;
  if (m > 256) return LN_ERR_UNSUPPORTED;
  if (ws_bytes < ns_pinv_workspace_bytes(batch, m, iters)) return LN_ERR_WORKSPACE;
  const NsWs w = carve_ns_ws(batch, m, iters, ws);
  launch_ns_pinv(batch, m, iters, ridge_eps, alpha, W, w, X_hist ? X_hist : w.Xh, X, resid, static_cast<cudaStream_t>(stream));
  return launch_ok();
}

int ns_pinv_bwd(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha,
                const float* X_hist, const float* dX, float* dW, void* ws, size_t ws_bytes, void* stream) {
  if (batch <= 0 || m <= 0 || iters < 0 || !W || !dX || !dW || !ws) return LN_ERR_ARG;
  if (!(ridge_eps >= 0.f) || !isfinite(ridge_eps) || !isfinite(alpha)) return LN_ERR_ARG;
  if (!aligned16(W) || !aligned16(dX) || !aligned16(dW) || !aligned16(X_hist) || !aligned16(ws)) return LN_ERR_ARG;
  if (m > 256) return LN_ERR_UNSUPPORTED;
  if (ws_bytes < ns_pinv_workspace_bytes(batch, m, iters)) return LN_ERR_WORKSPACE;
  const NsWs w = carve_ns_ws(batch, m, iters, ws);
  {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int cl = ns_cluster(m);
    auto go = [&](auto kern) {
      LN_LAUNCH("k_ns_pinv_bwd", st, launch_clustered(kern, batch * cl, cl, 0, st, m, iters, ridge_eps, alpha, W, w.Wr, w.P, w.Hm, w.Ga, w.Gb, w.Xh,
                                                      X_hist, w.hdr, dX, dW));
    };
    if (cl == 8) go(k_ns_pinv_bwd<8>); else if (cl == 4) go(k_ns_pinv_bwd<4>); else go(k_ns_pinv_bwd<1>);
  }
  return launch_ok();
}

// ------------------------------------------------------------------------------------------
// ns_pinv for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off the table: inside a serving loop whose
// memory pool was carved up at start-up and is fully committed, in a plug-in that is handed
// input and output pointers and nothing else, or under a framework that forbids allocator
// calls on its worker threads.  ns_pinv itself needs scratch (the ridge-shifted matrix, one
// product and the iterates), which such a caller has no way to provide.  This variant keeps
// that scratch in a fixed array that is part of the library image: every GPU that loads the
// library holds LN_STATIC_SCRATCH_BYTES of device memory for it until the process exits.
//
// In host code the name of a __device__ array is only a stand-in; the device address has to be
// asked for, once per device, with that device current.  The first call on a device does that.
// ------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticScratchBytes = LN_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
std::atomic<void*> g_static_scratch_addr[kMaxDevices];   // device address of g_static_scratch, per device; NULL = not asked yet

// Device address of the static scratch on the current device (looked up on first use).
int static_scratch_ptr(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LN_ERR_CUDA;
  void* ptr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (!ptr) {      // two threads may both ask; they get the same address
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return LN_ERR_CUDA;
    g_static_scratch_addr[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return LN_OK;
}
}  // namespace

size_t ns_pinv_static_scratch_bytes(void) { return kStaticScratchBytes; }

int ns_pinv_static(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha, float* X,
                   float* resid, void* stream) {
  if (batch <= 0 || m <= 0 || iters < 0 || !W || !X) return LN_ERR_ARG;
  if (!(ridge_eps >= 0.f) || !isfinite(ridge_eps) || !isfinite(alpha)) return LN_ERR_ARG;
  if (!aligned16(W) || !aligned16(X)) return LN_ERR_ARG;
  if (m > 256) return LN_ERR_UNSUPPORTED;
  if (ns_pinv_workspace_bytes(batch, m, iters) > kStaticScratchBytes) return LN_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  const int s = static_scratch_ptr(&scratch);
  if (s != LN_OK) return s;
  // Every piece of the scratch is written by the kernel before it is read, so the contents a
  // previous call left behind do not matter and nothing has to be cleared.
  const NsWs w = carve_ns_ws(batch, m, iters, scratch);
  launch_ns_pinv(batch, m, iters, ridge_eps, alpha, W, w, w.Xh, X, resid, static_cast<cudaStream_t>(stream));
  return launch_ok();
}

int l1_kernel(int32_t batch, int32_t na, int32_t nb, int32_t d, const void* A, const void* Bm, int32_t dtype,
              float lambda, float* Kout, float* rowsum, void* stream) {
  if (batch <= 0 || na <= 0 || nb <= 0 || d <= 0 || !A || !Bm || !Kout) return LN_ERR_ARG;
  if (!(lambda > 0.f) || !isfinite(lambda)) return LN_ERR_ARG;
  if (dtype != LN_F32 && dtype != LN_BF16) return LN_ERR_ARG;
  if (!aligned16(A) || !aligned16(Bm) || !aligned16(Kout) || !aligned16(rowsum)) return LN_ERR_ARG;
  if (batch > 65535) return LN_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == LN_F32) launch_l1<float, float>("l1_kernel", (const float*)A, (const float*)Bm, Kout, rowsum, batch, na, nb, d, nb, lambda, st);
  else launch_l1<bf16, bf16>("l1_kernel", (const bf16*)A, (const bf16*)Bm, Kout, rowsum, batch, na, nb, d, nb, lambda, st);
  return launch_ok();
}


size_t l1_kernel_bwd_workspace_bytes(int32_t batch, int32_t na, int32_t nb, int32_t d) {
  if (batch <= 0 || na <= 0 || nb <= 0 || d <= 0) return 0;
  return carve_l1bwd(batch, na, nb, d, nullptr).bytes;
}

int l1_kernel_bwd(int32_t batch, int32_t na, int32_t nb, int32_t d, const void* A, const void* Bm, int32_t dtype,
                  float lambda, const float* Kmat, const float* dKmat, void* dA, void* dB, void* ws, size_t ws_bytes,
                  void* stream) {
  if (batch <= 0 || na <= 0 || nb <= 0 || d <= 0 || !A || !Bm || !dKmat || !dA || !dB || !ws) return LN_ERR_ARG;
  if (!(lambda > 0.f) || !isfinite(lambda)) return LN_ERR_ARG;
  if (dtype != LN_F32 && dtype != LN_BF16) return LN_ERR_ARG;
  if (!aligned16(A) || !aligned16(Bm) || !aligned16(Kmat) || !aligned16(dKmat) || !aligned16(dA) || !aligned16(dB) ||
      !aligned16(ws))
    return LN_ERR_ARG;
  if (d != 32 && d != 64 && d != 128) return LN_ERR_UNSUPPORTED;
  if (batch > 65535) return LN_ERR_UNSUPPORTED;
  if (ws_bytes < l1_kernel_bwd_workspace_bytes(batch, na, nb, d)) return LN_ERR_WORKSPACE;
  const L1BwdWs w = carve_l1bwd(batch, na, nb, d, ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define LN_L1B(T, D) l1_bwd_impl<T, D>(batch, na, nb, (const T*)A, (const T*)Bm, lambda, Kmat, dKmat, (T*)dA, (T*)dB, w, st)
  if (dtype == LN_F32) { if (d == 32) LN_L1B(float, 32); else if (d == 64) LN_L1B(float, 64); else LN_L1B(float, 128); }
  else { if (d == 32) LN_L1B(bf16, 32); else if (d == 64) LN_L1B(bf16, 64); else LN_L1B(bf16, 128); }
#undef LN_L1B
  return launch_ok();
}

int landmarks_pool(const ln_problem* p, const void* K, float* L, void* stream) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (p->lm_mode < 1 || !K || !L || !aligned16(K) || !aligned16(L)) return LN_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (p->dtype == LN_F32) launch_pool<float>(p, (const float*)K, L, st);
  else launch_pool<bf16>(p, (const bf16*)K, L, st);
  return launch_ok();
}

int landmarks_pool_bwd(const ln_problem* p, const float* dL, void* dK, void* stream) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (p->lm_mode < 1 || !dL || !dK || !aligned16(dL) || !aligned16(dK)) return LN_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dim3 grid(cdiv((long long)p->n * (p->d / 4), 256 * POOL_EPT), p->B * p->H);
  if (p->dtype == LN_F32) LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<float><<<grid, 256, 0, st>>>(nullptr, dL, (float*)dK, geom_of(p), 1));
  else LN_LAUNCH("k_pool_bwd", st, k_pool_bwd<bf16><<<grid, 256, 0, st>>>(nullptr, dL, (bf16*)dK, geom_of(p), 1));
  return launch_ok();
}

int laplace_nystrom_saved_array(const ln_problem* p, const char* name, int64_t info[5]) {
  if (validate(p) != LN_OK || !name || !info) return LN_ERR_ARG;
  Plan pl; make_plan(p, &pl);
  const Ctx x = carve_ctx(pl, reinterpret_cast<void*>(256));      // offsets relative to a fictitious base
  auto off = [](const void* q) { return (int64_t)((reinterpret_cast<uintptr_t>(q) - 256) / sizeof(float)); };
  const int64_t n = p->n, d = p->d, m = p->m, ldm = pl.ldm;
  const bool img = p->dtype == LN_BF16 && !pl.two;                 // tcgen05 paths: history slots are operand images
  const int64_t ldx = (img && m <= 128) ? ldm : m;
  const int64_t mx = img ? pl.hslot : m * ldx;
  struct { const char* nm; const void* ptr; int64_t rows, cols, ld, stride; } t[] = {
    {"L", x.Lf, m, d, d, m * d}, {"C", x.C, n, m, ldm, n * ldm}, {"Rt", x.Rt, n, m, ldm, n * ldm},
    {"mu", x.mu, 1, n, n, n}, {"W", x.W, m, m, m, m * m},
    {"X", x.Xh + (size_t)pl.T * mx, m, m, ldx, (int64_t)(pl.T + 1) * mx},
    {"M", x.M, m, d, d, m * d}, {"Yt", x.Yt, m, d, d, m * d}, {"ybar", x.ybar, 1, d, d, d},
    {"Lq", x.Lq, m, d, d, m * d}};
  for (auto& e : t)
    if (strcmp(name, e.nm) == 0) {
      if (e.ptr == x.Lq && !pl.two) return LN_ERR_ARG;
      info[0] = off(e.ptr); info[1] = e.rows; info[2] = e.cols; info[3] = e.ld; info[4] = e.stride;
      return LN_OK;
    }
  return LN_ERR_ARG;
}

int ln_selftest_wait_timeout(int32_t probes, int32_t* dev_status, void* stream) {
  if (probes <= 0 || probes > (1 << 22) || !dev_status) return LN_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LN_LAUNCH("k_selftest_wait", st, k_selftest_wait<<<1, 32, 0, st>>>(probes, dev_status));
  return launch_ok();
}

int ln_fp32_add_probe(int32_t blocks, int32_t iters, int32_t mode, float* sink, void* stream) {
  if (blocks <= 0 || iters <= 0 || !sink || mode < 0 || mode > 5) return LN_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LN_LAUNCH("k_fp32_add_probe", st, k_fp32_add_probe<<<blocks, 256, 0, st>>>(iters, mode, sink));
  return launch_ok();
}
int64_t ln_fp32_add_probe_lane_ops(int32_t blocks, int32_t iters, int32_t mode) {
  const int per_step[6] = {2, 2, 6, 4, 6, 6};
  return (mode < 0 || mode > 5) ? 0 : (int64_t)blocks * 256 * iters * kProbeChains * per_step[mode];
}

// ------------------------------------------------------------------------------------------
// The attention block around the path: rotary embedding on Q and K, Nystrom Laplacian attention, + DWC(V)
// ------------------------------------------------------------------------------------------
}  // extern "C"
namespace {
int validate_block(const ln_problem* p, const ln_block* b) {
  int s = validate(p);
  if (s != LN_OK) return s;
  if (!b) return LN_ERR_ARG;
  if (p->lm_mode < 1) return LN_ERR_UNSUPPORTED;             // the token grid is needed
  if (!(b->rope_base >= 0.f) || !isfinite(b->rope_base)) return LN_ERR_ARG;
  if (b->rope_base > 0.f && (b->rope_base <= 1.f || (p->d & 3))) return LN_ERR_ARG;
  if (b->dwc_w && (b->dwc_ks < 1 || b->dwc_ks > 7 || (b->dwc_ks & 1) == 0 || !aligned16(b->dwc_w))) return LN_ERR_ARG;
  return LN_OK;
}
size_t tensor_bytes(const ln_problem* p) { return align_up((size_t)p->B * p->H * p->n * p->d * (p->dtype == LN_F32 ? 4 : 2), 256); }
// tokens per chunk of the filter-gradient partial sums: at least 512, at most 32 chunks per head
int dwc_tokens_per_chunk(const ln_problem* p) { const int g = p->gh * p->gw, t = (g + 31) / 32; return t < 512 ? 512 : t; }
int dwc_chunks(const ln_problem* p) { const int t = dwc_tokens_per_chunk(p); return (p->gh * p->gw + t - 1) / t; }
// rotation table of a call (at the end of the block workspace): one (cos, sin) pair of doubles per grid position and channel pair
size_t rope_table_bytes(const ln_problem* p) { return align_up((size_t)p->gh * p->gw * (p->d / 2) * sizeof(double2), 256); }
void launch_rope_table(const ln_problem* p, const ln_block* b, double2* tab, cudaStream_t st) {
  const long long cnt = (long long)p->gh * p->gw * (p->d / 2);
  LN_LAUNCH("rope_table", st, k_rope_table<<<cdiv(cnt, 256), 256, 0, st>>>(tab, cnt, p->d, log2((double)b->rope_base)));
}
template <typename T>
void launch_rope(const char* name, const ln_problem* p, const double2* tab, const void* X, void* out, double sign, cudaStream_t st) {
  // a thread per (token, channel quad) walks a share of the heads; shares so that about four CTAs per SM are launched
  const int BH = p->B * p->H, gx = (int)cdiv((long long)p->n * (p->d / 4), 256);
  int gy = (int)cdiv(4ll * sm_count(), gx); if (gy > BH) gy = BH; if (gy < 1) gy = 1;
  const int hpc = (BH + gy - 1) / gy; gy = (BH + hpc - 1) / hpc;
  LN_LAUNCH(name, st, k_rope<T><<<dim3(gx, gy), 256, 0, st>>>((const T*)X, (T*)out, BH, hpc, p->n, p->d, p->prefix, tab, sign));
}
// the tcgen05 product kernels (bf16 storage, 64 or 128 dims) take the convolution branch into their epilogue
inline bool dwc_in_epilogue(const ln_problem* p) { return p->dtype == LN_BF16 && (p->d == 64 || p->d == 128); }
template <typename T>
void launch_dwc_add(const char* name, const ln_problem* p, const ln_block* b, const void* src, void* out, int flip, cudaStream_t st) {
  LN_LAUNCH(name, st, k_dwc_add<T><<<dim3(cdiv((long long)p->gh * p->gw * (p->d / 4), 256), p->B * p->H), 256, 0, st>>>(
                (const T*)src, b->dwc_w, (T*)out, p->H, p->n, p->d, p->prefix, p->gh, p->gw, b->dwc_ks, flip));
}
}  // namespace
extern "C" {

size_t laplace_attention_block_saved_bytes(const ln_problem* p, const ln_block* b) {
  if (validate_block(p, b) != LN_OK) return 0;
  return laplace_nystrom_saved_bytes(p) + (b->rope_base > 0.f ? 2 * tensor_bytes(p) : 0);
}

size_t laplace_attention_block_workspace_bytes(const ln_problem* p, const ln_block* b) {
  if (validate_block(p, b) != LN_OK) return 0;
  size_t ws = laplace_nystrom_workspace_bytes(p, 1);
  if (b->rope_base > 0.f) ws += 2 * tensor_bytes(p);                           // gradients with respect to the rotated Q and K
  if (b->dwc_w) ws += align_up((size_t)p->B * p->H * dwc_chunks(p) * p->d * b->dwc_ks * b->dwc_ks * sizeof(float), 256);
  ws = align_up(ws, 256);
  if (b->rope_base > 0.f) ws += rope_table_bytes(p);                           // the rotation table, last
  return ws;
}

int laplace_attention_block_fwd(const ln_problem* p, const ln_block* b, const void* Q, const void* K, const void* V, void* O,
                                void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  int s = validate_block(p, b);
  if (s != LN_OK) return s;
  if (!Q || !K || !V || !O || !saved || !ws) return LN_ERR_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(saved) || !aligned16(ws)) return LN_ERR_ARG;
  if (ws_bytes < laplace_attention_block_workspace_bytes(p, b)) return LN_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t tb = tensor_bytes(p);
  char* sv = static_cast<char*>(saved);
  const void *q = Q, *k = K;
  void* inner_saved = sv;
  if (b->rope_base > 0.f) {
    s = check_fwd_args(p, sv, sv + tb, V, nullptr, O, sv + 2 * tb, ws, ws_bytes);
    if (s != LN_OK) return s;
    double2* tab = reinterpret_cast<double2*>(static_cast<char*>(ws) + laplace_attention_block_workspace_bytes(p, b) - rope_table_bytes(p));
    launch_rope_table(p, b, tab, st);
    if (p->dtype == LN_F32) { launch_rope<float>("rope_Q", p, tab, Q, sv, 1.f, st); launch_rope<float>("rope_K", p, tab, K, sv + tb, 1.f, st); }
    else { launch_rope<bf16>("rope_Q", p, tab, Q, sv, 1.f, st); launch_rope<bf16>("rope_K", p, tab, K, sv + tb, 1.f, st); }
    q = sv; k = sv + tb; inner_saved = sv + 2 * tb;
  }
  // the convolution branch rides in the epilogue of the O product where that product is the tcgen05 kernel; else its own pass
  const bool fused_dwc = b->dwc_w && dwc_in_epilogue(p);
  const DwcEpi epi = {V, b->dwc_w, p->H, p->prefix, p->gh, p->gw, b->dwc_ks, 0};
  s = fwd_entry(p, q, k, V, nullptr, O, inner_saved, ws, ws_bytes, dev_status, stream, true, fused_dwc ? &epi : nullptr);
  if (s != LN_OK) return s;
  if (b->dwc_w && !fused_dwc) {
    if (p->dtype == LN_F32) launch_dwc_add<float>("dwc_O", p, b, V, O, 0, st); else launch_dwc_add<bf16>("dwc_O", p, b, V, O, 0, st);
  }
  return launch_ok();
}

int laplace_attention_block_bwd(const ln_problem* p, const ln_block* b, const void* Q, const void* K, const void* V,
                                const void* dO, const void* saved, void* dQ, void* dK, void* dV, float* dWd, void* ws,
                                size_t ws_bytes, int32_t* dev_status, void* stream) {
  int s = validate_block(p, b);
  if (s != LN_OK) return s;
  if (!Q || !K || !V || !dO || !saved || !dQ || !dK || !dV || !ws) return LN_ERR_ARG;
  if ((b->dwc_w != nullptr) != (dWd != nullptr)) return LN_ERR_ARG;
  if (!aligned16(saved) || !aligned16(ws) || !aligned16(dWd)) return LN_ERR_ARG;
  if (ws_bytes < laplace_attention_block_workspace_bytes(p, b)) return LN_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t tb = tensor_bytes(p), base_ws = align_up(laplace_nystrom_workspace_bytes(p, 1), 256);
  const char* sv = static_cast<const char*>(saved);
  char* w = static_cast<char*>(ws);
  const bool rope = b->rope_base > 0.f;
  const void *q = rope ? (const void*)sv : Q, *k = rope ? (const void*)(sv + tb) : K;
  void *dq = rope ? (void*)(w + base_ws) : dQ, *dk = rope ? (void*)(w + base_ws + tb) : dK;
  float* wpart = reinterpret_cast<float*>(w + base_ws + (rope ? 2 * tb : 0));
  const bool fused_dwc = b->dwc_w && dwc_in_epilogue(p);
  const DwcEpi epi = {dO, b->dwc_w, p->H, p->prefix, p->gh, p->gw, b->dwc_ks, 1};
  s = bwd_entry(p, q, k, V, nullptr, dO, rope ? sv + 2 * tb : sv, dq, dk, dV, nullptr, ws, base_ws, dev_status, stream, true,
                fused_dwc ? &epi : nullptr);
  if (s != LN_OK) return s;
  if (rope) {
    double2* tab = reinterpret_cast<double2*>(w + laplace_attention_block_workspace_bytes(p, b) - rope_table_bytes(p));
    launch_rope_table(p, b, tab, st);
    if (p->dtype == LN_F32) { launch_rope<float>("rope_dQ", p, tab, dq, dQ, -1.f, st); launch_rope<float>("rope_dK", p, tab, dk, dK, -1.f, st); }
    else { launch_rope<bf16>("rope_dQ", p, tab, dq, dQ, -1.f, st); launch_rope<bf16>("rope_dK", p, tab, dk, dK, -1.f, st); }
  }
  if (b->dwc_w) {
    const int ch = dwc_chunks(p), BH = p->B * p->H, cnt = p->d * b->dwc_ks * b->dwc_ks;
    if (p->dtype == LN_F32) {
      launch_dwc_add<float>("dwc_dV", p, b, dO, dV, 1, st);
      if (b->dwc_ks == 3)
        LN_LAUNCH("dwc_wgrad", st, k_dwc_wgrad3<float><<<dim3(ch, BH), 256, 0, st>>>((const float*)V, (const float*)dO, wpart, p->n, p->d, p->prefix,
                                                                                     p->gh, p->gw, dwc_tokens_per_chunk(p)));
      else
      LN_LAUNCH("dwc_wgrad", st, k_dwc_wgrad<float><<<dim3(ch, BH, b->dwc_ks), 256, 0, st>>>((const float*)V, (const float*)dO, wpart, p->n, p->d, p->prefix,
                                                                                            p->gh, p->gw, b->dwc_ks, dwc_tokens_per_chunk(p)));
    } else {
      if (!fused_dwc) launch_dwc_add<bf16>("dwc_dV", p, b, dO, dV, 1, st);
      if (b->dwc_ks == 3)
        LN_LAUNCH("dwc_wgrad", st, k_dwc_wgrad3<bf16><<<dim3(ch, BH), 256, 0, st>>>((const bf16*)V, (const bf16*)dO, wpart, p->n, p->d, p->prefix,
                                                                                    p->gh, p->gw, dwc_tokens_per_chunk(p)));
      else
      LN_LAUNCH("dwc_wgrad", st, k_dwc_wgrad<bf16><<<dim3(ch, BH, b->dwc_ks), 256, 0, st>>>((const bf16*)V, (const bf16*)dO, wpart, p->n, p->d, p->prefix,
                                                                                           p->gh, p->gw, b->dwc_ks, dwc_tokens_per_chunk(p)));
    }
    LN_LAUNCH("dwc_wreduce", st, k_dwc_wreduce<<<dim3(cdiv(cnt, 128), p->H), 256, 0, st>>>(wpart, dWd, p->B, p->H, ch, cnt));
  }
  return launch_ok();
}

int laplace_exact_fwd(int32_t batch, int32_t n, int32_t d, int32_t dtype, float lambda, int32_t map_mode, const void* Q,
                      const void* K, const void* V, void* O, void* stream) {
  if (batch <= 0 || n <= 0 || !Q || !K || !V || !O) return LN_ERR_ARG;
  if (!(lambda > 0.f) || !isfinite(lambda) || (map_mode != 0 && map_mode != 1)) return LN_ERR_ARG;
  if (dtype != LN_F32 && dtype != LN_BF16) return LN_ERR_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return LN_ERR_ARG;
  if ((d != 32 && d != 64 && d != 128) || batch > 65535) return LN_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float nscale = -1.4426950408889634f / lambda;
  auto go = [&](auto kern, size_t smem) {
    want_smem(kern, smem);
    using TT = std::remove_const_t<std::remove_pointer_t<decltype(arg0(kern))>>;
    LN_LAUNCH("k_exact_fwd", st, kern<<<dim3(cdiv(n, 64), batch), 256, smem, st>>>((const TT*)Q, (const TT*)K, (const TT*)V, (TT*)O, n, nscale, map_mode));
  };
  if (dtype == LN_F32) { if (d == 32) go(k_exact_fwd<float, 32>, exact_smem_bytes<32>()); else if (d == 64) go(k_exact_fwd<float, 64>, exact_smem_bytes<64>()); else go(k_exact_fwd<float, 128>, exact_smem_bytes<128>()); }
  else { if (d == 32) go(k_exact_fwd<bf16, 32>, exact_smem_bytes<32>()); else if (d == 64) go(k_exact_fwd<bf16, 64>, exact_smem_bytes<64>()); else go(k_exact_fwd<bf16, 128>, exact_smem_bytes<128>()); }
  return launch_ok();
}

}  // extern "C"
