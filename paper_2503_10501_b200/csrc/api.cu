// C ABI of libtokencarve: argument checks, workspace planning, and the order in which the
// kernels of each stage are enqueued.
#include <math.h>
#include <string.h>

#include <atomic>
#include <functional>
#include <mutex>
#include <vector>

#include "tc_internal.cuh"

namespace tc {

static std::atomic<long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- optional event profile ---------------------------------------------------------------
struct Profiler {
  std::mutex mu;
  bool on = false;
  std::vector<cudaEvent_t> ev;   // pairs (start, stop)
  std::vector<int> cls;          // class of each pair
  std::vector<long long> launches_at_open, launches_at_close;
  size_t used = 0;               // pairs in use
};
static Profiler g_prof;

Scope::Scope(int cls, cudaStream_t s) : slot(-1), st(s) {
  if (!g_prof.on) return;
  std::lock_guard<std::mutex> lk(g_prof.mu);
  if (g_prof.used == g_prof.cls.size()) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
    g_prof.ev.push_back(a);
    g_prof.ev.push_back(b);
    g_prof.cls.push_back(cls);
    g_prof.launches_at_open.push_back(0);
    g_prof.launches_at_close.push_back(0);
  }
  slot = (int)g_prof.used++;
  g_prof.cls[slot] = cls;
  g_prof.launches_at_open[slot] = g_launches.load();
  cudaEventRecord(g_prof.ev[2 * slot], st);
}
Scope::~Scope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_prof.mu);
  cudaEventRecord(g_prof.ev[2 * slot + 1], st);
  g_prof.launches_at_close[slot] = g_launches.load();
}

tc_status launch_gram_simt(const Dims& D, const void* O, float* G, cudaStream_t st);
tc_status launch_gram_tc(const Dims& D, const void* O, float* G, int32_t* status, cudaStream_t st);
void fill_i32(int32_t* p, int n, int v, cudaStream_t st);

tc_status make_dims(const tc_params* p, Dims* out) {
  if (p == nullptr || out == nullptr) return TC_ERR_INVALID_ARG;
  Dims D;
  memset(&D, 0, sizeof(D));
  D.B = p->batch; D.N = p->n_tokens; D.d = p->d_model; D.H = p->n_heads; D.dh = p->head_dim;
  D.T = p->n_query; D.keep = p->keep;
  if (D.B < 1 || D.N < 1 || D.d < 1 || D.H < 1 || D.dh < 1 || D.T < 1) return TC_ERR_INVALID_ARG;
  if (D.keep < 1 || D.keep > D.N) return TC_ERR_INVALID_ARG;
  if (!(p->lambda >= 0.f && p->lambda <= 1.f)) return TC_ERR_INVALID_ARG;
  if (!(p->rank_tol >= 0.f && p->rank_tol < 1.f)) return TC_ERR_INVALID_ARG;
  if (p->dtype != TC_F16 && p->dtype != TC_F32 && p->dtype != TC_BF16) return TC_ERR_INVALID_ARG;
  if (p->score_norm != TC_NORM_NONE && p->score_norm != TC_NORM_SUM1) return TC_ERR_INVALID_ARG;
  if ((p->flags & ~(uint32_t)(TC_FLAG_SIM_MASK | TC_FLAG_WEIGHTED_MERGE)) != 0) return TC_ERR_INVALID_ARG;
  D.sim_src = (int)(p->flags & TC_FLAG_SIM_MASK);
  if (D.sim_src > 2) return TC_ERR_INVALID_ARG;
  D.wmerge = (p->flags & TC_FLAG_WEIGHTED_MERGE) != 0;
  // M = floor(L_vc * rho), P = L_vc + M (Sec. 3.3.1 / 3.3.2), Set A = first half (Eq. 3-9)
  int M;
  if (p->n_merge < 0) {
    if (!(p->rho >= 0.f && p->rho <= 1.f)) return TC_ERR_INVALID_ARG;
    M = (int)floor((double)D.keep * (double)p->rho);
  } else {
    M = p->n_merge;
  }
  if (M > D.N - D.keep) M = D.N - D.keep;
  if (M < 0) M = 0;
  D.M = M;
  D.P = D.keep + M;
  D.nA = D.P / 2;
  D.nB = D.P - D.nA;
  if (D.M > D.nB) return TC_ERR_INVALID_ARG;
  D.f16 = (p->dtype == TC_F16);
  D.bf16 = (p->dtype == TC_BF16);
  D.esz = (D.f16 || D.bf16) ? 2 : 4;
  // rows must be whole 16-byte vectors for the gather; selection kernels cover N <= 4096
  if (((size_t)D.d * D.esz) % 16 != 0 || ((size_t)D.dh * D.esz) % 16 != 0) return TC_ERR_UNSUPPORTED;
  if (D.N > 4096) return TC_ERR_UNSUPPORTED;
  if (p->rank_cap < 0) return TC_ERR_INVALID_ARG;
  D.full = (p->rank_cap == 0) || (p->rank_cap >= D.N);
  D.k = D.full ? D.N : p->rank_cap;
  if (D.k > 1024) return TC_ERR_UNSUPPORTED;  // Jacobi keeps at most 32 elements per lane
  if (!D.full && D.k < 16) return TC_ERR_INVALID_ARG;
  // the subspace solve runs its products on the tensor cores when the shapes fit its tiles
  // (the sign sketch keeps one row of signs, d floats, in shared memory)
  D.tcp = !D.full && (D.N & 3) == 0 && (size_t)D.d * sizeof(float) <= 48 * 1024 &&
          gemm_f32x3_supported(D.N, D.k, D.N) && gemm_f32x3_supported(D.N, D.k, D.k);
  D.max_sweeps = p->max_sweeps > 0 ? p->max_sweeps : 30;
  D.lambda = p->lambda;
  D.rank_tol = p->rank_tol;
  D.score_norm = p->score_norm;
  // row chunks of the attention reduction: sixteen blocks per SM when the rows allow it (the
  // blocks are not all the same length, so many short ones balance better than a few long
  // ones), at least 32 rows each
  const int R = D.H * D.T;
  int chunks = (16 * 148 + D.B - 1) / D.B;
  if (chunks > R / 32) chunks = R / 32;
  if (chunks > 64) chunks = 64;
  if (chunks < 1) chunks = 1;
  D.chunks = chunks;
  *out = D;
  return TC_OK;
}

Plan make_plan(const Dims& D) {
  Plan P;
  memset(&P, 0, sizeof(P));
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t B = D.B, N = D.N, k = D.k;
  P.s_part = take(B * D.chunks * N * 4);
  P.S = take(B * N * 4);
  P.C = take(B * N * 4);
  P.E = take(B * N * 4);
  P.sigma = take(B * k * 4);
  P.G = take(B * N * N * 4);
  if (D.tcp) {
    P.panel_T_off = align_up(B * N * k * 4, 256);
    P.PA = take(2 * P.panel_T_off);
    P.PB = take(2 * P.panel_T_off);
    P.Sk = take(B * k * k * 4);
    P.Hk = take(B * k * k * 4);
    P.Rinv = take(B * k * k * 4);
    P.Es = take(B * 4 * k * k * 4);
  } else if (!D.full) {
    P.Y0 = take(B * N * k * 4);
    P.Y1 = take(B * N * k * 4);
    P.Y2 = take(B * N * k * 4);
    const size_t parts = (size_t)tn_parts(D.k);  // k x k products arrive in this many parts
    P.Sm = take(B * k * k * 4 * parts);
    P.Rinv = take(B * k * k * 4);
    P.Hm = take(B * k * k * 4 * parts);
  }
  if (!D.tcp) {
    P.W = take(B * k * k * 4);
    P.ZT = take(B * k * k * 4);
  }
  P.setA = take(B * (size_t)(D.nA > 0 ? D.nA : 1) * 4);
  P.setB = take(B * (size_t)D.nB * 4);
  P.best_val = take(B * (size_t)D.nB * 4);
  P.best_dst = take(B * (size_t)D.nB * 4);
  P.msrc = take(B * (size_t)(D.M > 0 ? D.M : 1) * 4);
  P.mdst = take(B * (size_t)(D.M > 0 ? D.M : 1) * 4);
  P.kept = take(B * (size_t)D.keep * 4);
  P.rank = take(B * 4);
  P.flags = take(B * 4);
  if (D.sim_src == 2) P.Kmean = take(B * N * (size_t)D.dh * 4);
  P.total = off;
  return P;
}

// float16 inputs go to the tensor cores; float32 inputs keep full precision on the plain ALUs
tc_status launch_gram(const Dims& D, const void* O, float* G, int32_t* status, cudaStream_t st) {
  if (D.f16 || D.bf16) return launch_gram_tc(D, O, G, status, st);
  return launch_gram_simt(D, O, G, st);
}

static tc_status check_launch() {
  return cudaGetLastError() == cudaSuccess ? TC_OK : TC_ERR_CUDA;
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

struct Ctx {
  Dims D;
  Plan P;
  char* ws;
  cudaStream_t st;
};

static tc_status open_ctx(const tc_params* p, void* ws, size_t ws_bytes, void* stream, Ctx* c) {
  tc_status s = make_dims(p, &c->D);
  if (s != TC_OK) return s;
  c->P = make_plan(c->D);
  if (ws == nullptr || misaligned(ws)) return TC_ERR_INVALID_ARG;
  if (ws_bytes < c->P.total) return TC_ERR_WORKSPACE;
  c->ws = (char*)ws;
  c->st = (cudaStream_t)stream;
  return TC_OK;
}

// ---- concurrent image groups ----------------------------------------------------------------
// The Cholesky and eigen-solver kernels run one block per image and so leave most of the GPU
// idle at batch sizes below the SM count.  The batch is therefore cut into a few groups whose
// Gram -> eigen-solve chains run on separate internal streams, forked from and joined back into
// the caller's stream with events: one group's single-block kernels overlap another group's
// GEMMs.  Per-image results do not depend on the grouping.
constexpr int kMaxGroups = 16;
struct GroupStreams {
  bool ready = false;
  cudaStream_t s[kMaxGroups];    // a group's sketch -> Cholesky-QR -> eigen-solve chain
  cudaStream_t s2[kMaxGroups];   // its Gram matrix, which the chain needs only from G Q on
  cudaEvent_t fork, join[kMaxGroups], gram_done[kMaxGroups];
  cudaEvent_t attn_done;         // the attention partial sums of the whole batch are written
};
static std::mutex g_groups_mu;
static GroupStreams g_groups[64];
static std::atomic<int> g_n_groups{4};

static GroupStreams* group_streams() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  GroupStreams& g = g_groups[dev];
  if (!g.ready) {
    for (int i = 0; i < kMaxGroups; ++i) {
      if (cudaStreamCreateWithFlags(&g.s[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
      if (cudaStreamCreateWithFlags(&g.s2[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&g.join[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&g.gram_done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    if (cudaEventCreateWithFlags(&g.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&g.attn_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    g.ready = true;
  }
  return &g;
}

// score: S partial sums || (Gram -> eigen-solve -> C per image group) -> E
// A launcher that refuses (tensor map, function attribute) stops the enqueue: the group streams
// forked so far are joined back, the status words of the images not reached are set, and the
// caller gets the status.
// tail: what follows the scores of an image group on that group's stream (images b0 .. b0 + Dg.B),
// so that one group's selection and gather run beside another group's eigen-solve; null for none.
using GroupTail = std::function<void(const Dims& Dg, int b0, cudaStream_t st)>;
static tc_status enqueue_score(const Ctx& c, const void* O, const void* A, float* E, float* C, float* S,
                               float* sigma, int32_t* rank, int32_t* img_status,
                               const GroupTail* tail = nullptr) {
  const Dims& D = c.D;
  const int q = D.N < D.d ? D.N : D.d;
  fill_i32(img_status, D.B, 0, c.st);
  int ng = g_n_groups.load();
  if (ng > D.B) ng = D.B;
  std::lock_guard<std::mutex> lk(g_groups_mu);
  GroupStreams* gs = ng > 1 ? group_streams() : nullptr;
  if (gs == nullptr) ng = 1;
  if (ng > 1) cudaEventRecord(gs->fork, c.st);
  launch_attn_colsum(D, A, (float*)(c.ws + c.P.s_part), c.st);
  const bool group_tail = (tail != nullptr) && ng > 1;
  if (group_tail) cudaEventRecord(gs->attn_done, c.st);
  const int base = D.B / ng, extra = D.B % ng;
  int b0 = 0;
  tc_status err = TC_OK;
  for (int g = 0; g < ng && err == TC_OK; ++g) {
    const int nb = base + (g < extra ? 1 : 0);
    cudaStream_t st = ng > 1 ? gs->s[g] : c.st;
    if (ng > 1) cudaStreamWaitEvent(st, gs->fork, 0);
    // The groups start in up to four waves, a wave's Gram products behind those of the wave
    // before it: groups that all sit in the same phase of the chain compete for the same unit
    // (the tensor pipes in the products, 64 of 148 SMs in the single-block kernels) while the
    // others idle.  Measured at 64 images: 1.35 ms per carve in one wave, 1.29 ms in four.
    // (Under 32 images the kernels of different groups hardly compete and a wave only waits.)
    const int waves = D.B < 32 ? 1 : (ng >= 8 ? 4 : (ng >= 4 ? 2 : 1));
    const int per_wave = (ng + waves - 1) / waves;
    const bool late = (waves > 1) && (g >= per_wave) && !D.full;
    if (late) cudaStreamWaitEvent(st, gs->gram_done[g - per_wave], 0);
    Dims Dg = D;
    Dg.B = nb;
    const char* Og = (const char*)O + (size_t)b0 * D.N * D.d * D.esz;
    // the sketch and its first Cholesky-QR pass do not read G: with groups, the Gram matrix is
    // built beside them on a stream of its own and joined in front of the first product with G
    cudaEvent_t gram_done = nullptr;
    float* Gg = (float*)(c.ws + c.P.G) + (size_t)b0 * D.N * D.N;
    if (ng > 1 && !D.full) {
      cudaStreamWaitEvent(gs->s2[g], gs->fork, 0);
      if (late) cudaStreamWaitEvent(gs->s2[g], gs->gram_done[g - per_wave], 0);
      err = launch_gram(Dg, Og, Gg, img_status + b0, gs->s2[g]);
      cudaEventRecord(gs->gram_done[g], gs->s2[g]);
      gram_done = gs->gram_done[g];
    } else {
      err = launch_gram(Dg, Og, Gg, img_status + b0, st);
    }
    if (err == TC_OK)
      err = launch_ics(Dg, c.P, c.ws, b0, Og, C + (size_t)b0 * D.N, sigma ? sigma + (size_t)b0 * q : nullptr,
                       rank ? rank + b0 : nullptr, img_status + b0, st, nullptr, gram_done);
    else if (gram_done)
      cudaStreamWaitEvent(st, gram_done, 0);  // the side stream still joins the group's stream
    if (group_tail && err == TC_OK) {
      cudaStreamWaitEvent(st, gs->attn_done, 0);
      const size_t o = (size_t)b0 * D.N;
      launch_combine(Dg, (const float*)(c.ws + c.P.s_part) + o * D.chunks, C + o, S + o, E + o, st);
      (*tail)(Dg, b0, st);
    }
    if (ng > 1) {
      cudaEventRecord(gs->join[g], st);
      cudaStreamWaitEvent(c.st, gs->join[g], 0);
    }
    if (err != TC_OK) fill_i32(img_status + b0, D.B - b0, (int)err, c.st);
    b0 += nb;
  }
  if (err != TC_OK) return err;
  if (!group_tail) {
    launch_combine(D, (const float*)(c.ws + c.P.s_part), C, S, E, c.st);
    if (tail) (*tail)(D, 0, c.st);
  }
  return TC_OK;
}

}  // namespace tc

using namespace tc;

extern "C" {

tc_status tc_counts(const tc_params* p, int32_t* M, int32_t* P, int32_t* nA, int32_t* nB) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (M) *M = D.M;
  if (P) *P = D.P;
  if (nA) *nA = D.nA;
  if (nB) *nB = D.nB;
  return TC_OK;
}

tc_status tc_workspace_bytes(const tc_params* p, size_t* bytes) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (bytes == nullptr) return TC_ERR_INVALID_ARG;
  *bytes = make_plan(D).total;
  return TC_OK;
}

tc_status tc_score(const tc_params* p, const void* O, const void* A, float* E, float* C, float* S,
                   float* sigma, int32_t* rank, int32_t* img_status, void* ws, size_t ws_bytes,
                   void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, ws, ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  if (!O || !A || !E || !img_status || misaligned(O) || misaligned(A)) return TC_ERR_INVALID_ARG;
  float* Cw = C ? C : (float*)(c.ws + c.P.C);
  float* Sw = S ? S : (float*)(c.ws + c.P.S);
  s = enqueue_score(c, O, A, E, Cw, Sw, sigma, rank, img_status);
  if (s != TC_OK) return s;
  return check_launch();
}

tc_status tc_prune(const tc_params* p, const float* E, int32_t* setA, int32_t* setB, void* ws,
                   size_t ws_bytes, void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, ws, ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  if (!E || !setB || (c.D.nA > 0 && !setA)) return TC_ERR_INVALID_ARG;
  launch_prune(c.D, E, setA, setB, c.st);
  return check_launch();
}

tc_status tc_merge(const tc_params* p, const void* O, const int32_t* setA, const int32_t* setB,
                   int32_t* merge_src, int32_t* merge_dst, int32_t* kept_idx, void* ws,
                   size_t ws_bytes, void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, ws, ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  const Dims& D = c.D;
  if (!O || !setB || !kept_idx || (D.nA > 0 && !setA) || misaligned(O)) return TC_ERR_INVALID_ARG;
  if (D.M > 0 && (!merge_src || !merge_dst)) return TC_ERR_INVALID_ARG;
  if ((size_t)D.d * sizeof(float) > 48 * 1024) return TC_ERR_UNSUPPORTED;
  float* bv = (float*)(c.ws + c.P.best_val);
  int32_t* bd = (int32_t*)(c.ws + c.P.best_dst);
  int32_t* flags = (int32_t*)(c.ws + c.P.flags);
  fill_i32(flags, D.B, 0, c.st);
  if (D.M > 0) {
    if (D.sim_src == 2) {
      // the features are the head-mean keys: `O` is K [B, H, N, dh]
      float* Km = (float*)(c.ws + c.P.Kmean);
      launch_mean_heads(D, O, Km, c.st);
      launch_match_rows_f32(D, Km, D.dh, setA, setB, bv, bd, flags, c.st);
    } else {
      launch_match_rows(D, O, setA, setB, bv, bd, flags, c.st);  // rows of O, or of X
    }
  }
  launch_merge_select(D, setA, setB, bv, bd, merge_src, merge_dst, kept_idx, flags, c.st);
  return check_launch();
}

static tc_status compact_impl(const tc_params* p, const void* X, const void* K, const void* V,
                              const int32_t* kept_idx, const int32_t* merge_src,
                              const int32_t* merge_dst, const float* E, void* Xo, void* Ko,
                              void* Vo, void* ws, size_t ws_bytes, void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, ws, ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  const Dims& D = c.D;
  if (!X || !Xo || !kept_idx || misaligned(X) || misaligned(Xo)) return TC_ERR_INVALID_ARG;
  if (D.M > 0 && (!merge_src || !merge_dst)) return TC_ERR_INVALID_ARG;
  const bool kv = (K != nullptr);
  if (kv != (V != nullptr) || kv != (Ko != nullptr) || kv != (Vo != nullptr)) return TC_ERR_INVALID_ARG;
  if (kv && (misaligned(K) || misaligned(V) || misaligned(Ko) || misaligned(Vo))) return TC_ERR_INVALID_ARG;
  int32_t* flags = (int32_t*)(c.ws + c.P.flags);
  fill_i32(flags, D.B, 0, c.st);
  launch_compact(D, X, K, V, kept_idx, merge_src, merge_dst, Xo, Ko, Vo, E, flags, c.st);
  return check_launch();
}

tc_status tc_compact(const tc_params* p, const void* X, const void* K, const void* V,
                     const int32_t* kept_idx, const int32_t* merge_src, const int32_t* merge_dst,
                     void* Xo, void* Ko, void* Vo, void* ws, size_t ws_bytes, void* stream) {
  return compact_impl(p, X, K, V, kept_idx, merge_src, merge_dst, nullptr, Xo, Ko, Vo, ws, ws_bytes,
                      stream);
}

tc_status tc_compact_weighted(const tc_params* p, const void* X, const void* K, const void* V,
                              const int32_t* kept_idx, const int32_t* merge_src,
                              const int32_t* merge_dst, const float* E, void* Xo, void* Ko,
                              void* Vo, void* ws, size_t ws_bytes, void* stream) {
  if (E == nullptr) return TC_ERR_INVALID_ARG;
  return compact_impl(p, X, K, V, kept_idx, merge_src, merge_dst, E, Xo, Ko, Vo, ws, ws_bytes, stream);
}

tc_status tc_stage_status(const tc_params* p, const void* ws, size_t ws_bytes, int32_t* img_status,
                          void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, const_cast<void*>(ws), ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  if (!img_status) return TC_ERR_INVALID_ARG;
  if (cudaMemcpyAsync(img_status, c.ws + c.P.flags, (size_t)c.D.B * sizeof(int32_t),
                      cudaMemcpyDeviceToDevice, c.st) != cudaSuccess)
    return TC_ERR_CUDA;
  return TC_OK;
}

tc_status tc_carve(const tc_params* p, const void* O, const void* A, const void* X, const void* K,
                   const void* V, void* Xo, void* Ko, void* Vo, int32_t* kept_idx,
                   int32_t* img_status, void* ws, size_t ws_bytes, void* stream) {
  Ctx c;
  tc_status s = open_ctx(p, ws, ws_bytes, stream, &c);
  if (s != TC_OK) return s;
  const Dims& D = c.D;
  if (!O || !A || !X || !Xo || !kept_idx || !img_status) return TC_ERR_INVALID_ARG;
  if (misaligned(O) || misaligned(A) || misaligned(X) || misaligned(Xo)) return TC_ERR_INVALID_ARG;
  const bool kv = (K != nullptr);
  if (kv != (V != nullptr) || kv != (Ko != nullptr) || kv != (Vo != nullptr)) return TC_ERR_INVALID_ARG;
  if (kv && (misaligned(K) || misaligned(V) || misaligned(Ko) || misaligned(Vo))) return TC_ERR_INVALID_ARG;
  if (D.sim_src == 2 && !kv) return TC_ERR_INVALID_ARG;  // the head-mean keys need K
  if (D.sim_src != 0 && (size_t)(D.sim_src == 1 ? D.d : D.dh) * sizeof(float) > 48 * 1024)
    return TC_ERR_UNSUPPORTED;
  float* E = (float*)(c.ws + c.P.E);
  float* C = (float*)(c.ws + c.P.C);
  float* S = (float*)(c.ws + c.P.S);
  int32_t* setA = (int32_t*)(c.ws + c.P.setA);
  int32_t* setB = (int32_t*)(c.ws + c.P.setB);
  float* bv = (float*)(c.ws + c.P.best_val);
  int32_t* bd = (int32_t*)(c.ws + c.P.best_dst);
  int32_t* msrc = (int32_t*)(c.ws + c.P.msrc);
  int32_t* mdst = (int32_t*)(c.ws + c.P.mdst);
  // selection and gather of images b0 .. b0 + Dg.B on the stream their scores were computed on
  const GroupTail tail = [&](const Dims& Dg, int b0, cudaStream_t st) {
    const size_t b = (size_t)b0, esz = D.esz;
    const size_t kv_in = (size_t)D.H * D.N * D.dh * esz, kv_out = (size_t)D.H * D.keep * D.dh * esz;
    int32_t* sA = setA + b * D.nA;
    int32_t* sB = setB + b * D.nB;
    float* gbv = bv + b * D.nB;
    int32_t* gbd = bd + b * D.nB;
    int32_t* gst = img_status + b0;
    const char* Xg = (const char*)X + b * D.N * D.d * esz;
    const char* Kg = kv ? (const char*)K + b * kv_in : nullptr;
    const char* Vg = kv ? (const char*)V + b * kv_in : nullptr;
    launch_prune(Dg, E + b * D.N, sA, sB, st);
    if (D.M > 0) {
      if (D.sim_src == 0) {
        launch_match_gram(Dg, (const float*)(c.ws + c.P.G) + b * D.N * D.N, sA, sB, gbv, gbd, gst, st);
      } else if (D.sim_src == 1) {
        launch_match_rows(Dg, Xg, sA, sB, gbv, gbd, gst, st);
      } else {
        float* Km = (float*)(c.ws + c.P.Kmean) + b * D.N * D.dh;
        launch_mean_heads(Dg, Kg, Km, st);
        launch_match_rows_f32(Dg, Km, D.dh, sA, sB, gbv, gbd, gst, st);
      }
    }
    int32_t* gms = msrc + b * D.M;
    int32_t* gmd = mdst + b * D.M;
    int32_t* gk = kept_idx + b * D.keep;
    launch_merge_select(Dg, sA, sB, gbv, gbd, gms, gmd, gk, gst, st);
    launch_compact(Dg, Xg, Kg, Vg, gk, gms, gmd, (char*)Xo + b * D.keep * D.d * esz,
                   kv ? (char*)Ko + b * kv_out : nullptr, kv ? (char*)Vo + b * kv_out : nullptr,
                   D.wmerge ? E + b * D.N : nullptr, gst, st);
  };
  s = enqueue_score(c, O, A, E, C, S, nullptr, nullptr, img_status, &tail);
  if (s != TC_OK) return s;
  return check_launch();
}

// ---- host-buffer variant: device staging lives at the front of the workspace ---------------
constexpr int kHostChunks = 4;
struct HostStreams {
  bool ready = false;
  cudaStream_t cin, cout;
  cudaEvent_t fork, out, in[kHostChunks], done[kHostChunks];
};
static std::mutex g_host_mu;
static HostStreams g_host[64];

// scratch that covers the whole batch in one call as well as any of the chunks it is cut into
static size_t host_scratch_bytes(const tc_params* p, const Dims& D) {
  size_t need = make_plan(D).total;
  const int nchunk = D.B < kHostChunks ? D.B : kHostChunks;
  tc_params pc = *p;
  pc.batch = (D.B + nchunk - 1) / nchunk;
  Dims Dc;
  if (make_dims(&pc, &Dc) == TC_OK) {
    const size_t c = make_plan(Dc).total;
    if (c > need) need = c;
  }
  if (D.B / nchunk >= 1 && D.B / nchunk != pc.batch) {
    pc.batch = D.B / nchunk;
    if (make_dims(&pc, &Dc) == TC_OK) {
      const size_t c = make_plan(Dc).total;
      if (c > need) need = c;
    }
  }
  return need;
}

static HostStreams* host_streams() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostStreams& h = g_host[dev];
  if (!h.ready) {
    if (cudaStreamCreateWithFlags(&h.cin, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&h.cout, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&h.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&h.out, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < kHostChunks; ++i) {
      if (cudaEventCreateWithFlags(&h.in[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&h.done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    h.ready = true;
  }
  return &h;
}

struct HostPlan {
  size_t O, A, X, K, V, Xo, Ko, Vo, kept, status, scratch, total;
};

static HostPlan make_host_plan(const Dims& D, size_t scratch_bytes) {
  HostPlan h;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t B = D.B, e = D.esz;
  h.O = take(B * D.N * D.d * e);
  h.A = take(B * D.H * D.T * (size_t)D.N * e);
  h.X = take(B * D.N * D.d * e);
  h.K = take(B * D.H * D.N * (size_t)D.dh * e);
  h.V = take(B * D.H * D.N * (size_t)D.dh * e);
  h.Xo = take(B * D.keep * (size_t)D.d * e);
  h.Ko = take(B * D.H * D.keep * (size_t)D.dh * e);
  h.Vo = take(B * D.H * D.keep * (size_t)D.dh * e);
  h.kept = take(B * D.keep * 4);
  h.status = take(B * 4);
  h.scratch = off;
  h.total = off + scratch_bytes;
  return h;
}

tc_status tc_workspace_bytes_host(const tc_params* p, size_t* bytes) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (bytes == nullptr) return TC_ERR_INVALID_ARG;
  *bytes = make_host_plan(D, host_scratch_bytes(p, D)).total;
  return TC_OK;
}

tc_status tc_carve_host(const tc_params* p, const void* O, const void* A, const void* X,
                        const void* K, const void* V, void* Xo, void* Ko, void* Vo,
                        int32_t* kept_idx, int32_t* img_status, void* ws, size_t ws_bytes,
                        void* stream) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  const size_t scratch = host_scratch_bytes(p, D);
  HostPlan h = make_host_plan(D, scratch);
  if (ws == nullptr || misaligned(ws)) return TC_ERR_INVALID_ARG;
  if (ws_bytes < h.total) return TC_ERR_WORKSPACE;
  if (!O || !A || !X || !Xo || !kept_idx || !img_status) return TC_ERR_INVALID_ARG;
  const bool kv = (K != nullptr);
  if (kv != (V != nullptr) || kv != (Ko != nullptr) || kv != (Vo != nullptr)) return TC_ERR_INVALID_ARG;
  char* w = (char*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t e = D.esz;
  // bytes per image
  const size_t iO = (size_t)D.N * D.d * e, iA = (size_t)D.H * D.T * D.N * e;
  const size_t iKV = (size_t)D.H * D.N * D.dh * e;
  const size_t iXo = (size_t)D.keep * D.d * e, iKVo = (size_t)D.H * D.keep * D.dh * e;
  // The batch goes through in a few chunks: the upload of chunk c + 1 (copy-in stream) and the
  // download of chunk c - 1 (copy-out stream) run while chunk c is carved on `stream`.
  std::lock_guard<std::mutex> lk(g_host_mu);
  HostStreams* hs = host_streams();
  const int nchunk = (hs == nullptr) ? 1 : (D.B < kHostChunks ? D.B : kHostChunks);
  cudaStream_t cin = nchunk > 1 ? hs->cin : st, cout = nchunk > 1 ? hs->cout : st;
  bool ok = true;
  if (nchunk > 1) {
    ok &= cudaEventRecord(hs->fork, st) == cudaSuccess;
    ok &= cudaStreamWaitEvent(cin, hs->fork, 0) == cudaSuccess;
    ok &= cudaStreamWaitEvent(cout, hs->fork, 0) == cudaSuccess;
  }
  const int base = D.B / nchunk, extra = D.B % nchunk;
  int b0 = 0;
  for (int c = 0; c < nchunk; ++c) {
    const size_t nb = base + (c < extra ? 1 : 0), o = b0;
    ok &= cudaMemcpyAsync(w + h.O + o * iO, (const char*)O + o * iO, nb * iO, cudaMemcpyHostToDevice, cin) == cudaSuccess;
    ok &= cudaMemcpyAsync(w + h.A + o * iA, (const char*)A + o * iA, nb * iA, cudaMemcpyHostToDevice, cin) == cudaSuccess;
    ok &= cudaMemcpyAsync(w + h.X + o * iO, (const char*)X + o * iO, nb * iO, cudaMemcpyHostToDevice, cin) == cudaSuccess;
    if (kv) {
      ok &= cudaMemcpyAsync(w + h.K + o * iKV, (const char*)K + o * iKV, nb * iKV, cudaMemcpyHostToDevice, cin) == cudaSuccess;
      ok &= cudaMemcpyAsync(w + h.V + o * iKV, (const char*)V + o * iKV, nb * iKV, cudaMemcpyHostToDevice, cin) == cudaSuccess;
    }
    if (nchunk > 1) ok &= cudaEventRecord(hs->in[c], cin) == cudaSuccess;
    b0 += (int)nb;
  }
  if (!ok) return TC_ERR_CUDA;
  b0 = 0;
  for (int c = 0; c < nchunk; ++c) {
    const size_t nb = base + (c < extra ? 1 : 0), o = b0;
    if (nchunk > 1) ok &= cudaStreamWaitEvent(st, hs->in[c], 0) == cudaSuccess;
    tc_params pc = *p;
    pc.batch = (int32_t)nb;
    s = tc_carve(&pc, w + h.O + o * iO, w + h.A + o * iA, w + h.X + o * iO,
                 kv ? w + h.K + o * iKV : nullptr, kv ? w + h.V + o * iKV : nullptr,
                 w + h.Xo + o * iXo, kv ? w + h.Ko + o * iKVo : nullptr,
                 kv ? w + h.Vo + o * iKVo : nullptr, (int32_t*)(w + h.kept) + o * D.keep,
                 (int32_t*)(w + h.status) + o, w + h.scratch, scratch, stream);
    if (s != TC_OK) return s;
    if (nchunk > 1) {
      ok &= cudaEventRecord(hs->done[c], st) == cudaSuccess;
      ok &= cudaStreamWaitEvent(cout, hs->done[c], 0) == cudaSuccess;
    }
    ok &= cudaMemcpyAsync((char*)Xo + o * iXo, w + h.Xo + o * iXo, nb * iXo, cudaMemcpyDeviceToHost, cout) == cudaSuccess;
    if (kv) {
      ok &= cudaMemcpyAsync((char*)Ko + o * iKVo, w + h.Ko + o * iKVo, nb * iKVo, cudaMemcpyDeviceToHost, cout) == cudaSuccess;
      ok &= cudaMemcpyAsync((char*)Vo + o * iKVo, w + h.Vo + o * iKVo, nb * iKVo, cudaMemcpyDeviceToHost, cout) == cudaSuccess;
    }
    ok &= cudaMemcpyAsync(kept_idx + o * D.keep, (int32_t*)(w + h.kept) + o * D.keep, nb * D.keep * 4, cudaMemcpyDeviceToHost, cout) == cudaSuccess;
    ok &= cudaMemcpyAsync(img_status + o, (int32_t*)(w + h.status) + o, nb * 4, cudaMemcpyDeviceToHost, cout) == cudaSuccess;
    b0 += (int)nb;
  }
  if (nchunk > 1) {
    ok &= cudaEventRecord(hs->out, cout) == cudaSuccess;
    ok &= cudaStreamWaitEvent(st, hs->out, 0) == cudaSuccess;
  }
  return ok ? TC_OK : TC_ERR_CUDA;
}

tc_status tc_gram(const tc_params* p, const void* O, float* G, void* stream) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (!O || !G || misaligned(O) || misaligned(G)) return TC_ERR_INVALID_ARG;
  s = launch_gram(D, O, G, nullptr, (cudaStream_t)stream);
  if (s != TC_OK) return s;
  return check_launch();
}

tc_status tc_matmul_f32x3(const float* A, const float* B, float* C, float* CT, int32_t batch,
                          int32_t M, int32_t NN, int32_t K, int32_t* img_status, void* stream) {
  if (!A || !B || (!C && !CT) || batch < 1 || M < 1 || NN < 1 || K < 1) return TC_ERR_INVALID_ARG;
  if (misaligned(A) || misaligned(B) || (C && misaligned(C)) || (CT && misaligned(CT)))
    return TC_ERR_INVALID_ARG;
  if (!gemm_f32x3_supported(M, NN, K)) return TC_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  if (img_status) fill_i32(img_status, batch, 0, st);
  tc_status s = launch_gemm_f32x3(A, B, M, NN, K, batch, C, CT, img_status, st, KC_GEMM);
  if (s != TC_OK) return s;
  return check_launch();
}

// ---- Sec. 3.2: information quantity (numerical rank) of a set of tokens -----------------------
// The score path's own Gram and eigen kernels on the gathered rows.
// beyond the score path's own plan: the gathered rows, and four n x n arrays per image for the
// tridiagonal solver when the full problem is small enough for it
static size_t rank_rows_bytes(const Dims& D) { return align_up((size_t)D.B * D.N * D.d * D.esz, 256); }
static bool rank_small_full(const Dims& D) { return D.full && D.N <= 224; }
static size_t rank_extra_bytes(const Dims& D) {
  return rank_rows_bytes(D) + (rank_small_full(D) ? 4 * (size_t)D.B * D.N * D.N * sizeof(float) : 0);
}

static tc_status rank_dims(const tc_params* p, int32_t n_sub, Dims* full, Dims* sub) {
  if (p == nullptr) return TC_ERR_INVALID_ARG;
  tc_params pf = *p;  // the carve counts play no part here
  pf.keep = 1;
  pf.n_merge = 0;
  tc_status s = make_dims(&pf, full);
  if (s != TC_OK) return s;
  if (n_sub < 1 || n_sub > full->N) return TC_ERR_INVALID_ARG;
  pf.n_tokens = n_sub;
  return make_dims(&pf, sub);
}

tc_status tc_rank_workspace_bytes(const tc_params* p, int32_t n_sub, size_t* bytes) {
  Dims F, D;
  tc_status s = rank_dims(p, n_sub, &F, &D);
  if (s != TC_OK) return s;
  if (bytes == nullptr) return TC_ERR_INVALID_ARG;
  const Plan P = make_plan(D);
  *bytes = align_up(P.total, 256) + rank_extra_bytes(D);
  return TC_OK;
}

tc_status tc_rank(const tc_params* p, const void* O, const int32_t* idx, int32_t n_sub,
                  float* sigma, int32_t* rank, int32_t* img_status, void* ws, size_t ws_bytes,
                  void* stream) {
  Dims F, D;
  tc_status s = rank_dims(p, n_sub, &F, &D);
  if (s != TC_OK) return s;
  if (!O || !rank || !img_status || !ws || misaligned(O) || misaligned(ws)) return TC_ERR_INVALID_ARG;
  if (idx == nullptr && n_sub != F.N) return TC_ERR_INVALID_ARG;
  const Plan P = make_plan(D);
  const size_t rows_off = align_up(P.total, 256);
  if (ws_bytes < rows_off + rank_extra_bytes(D)) return TC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* w = (char*)ws;
  fill_i32(img_status, D.B, 0, st);
  const void* rows = O;
  if (idx != nullptr) {
    launch_gather_rows(F, n_sub, O, idx, w + rows_off, img_status, st);
    rows = w + rows_off;
  }
  s = launch_gram(D, rows, (float*)(w + P.G), img_status, st);
  if (s != TC_OK) return s;
  s = launch_ics(D, P, w, 0, rows, (float*)(w + P.C), sigma, rank, img_status, st,
                 rank_small_full(D) ? (float*)(w + rows_off + rank_rows_bytes(D)) : nullptr);
  if (s != TC_OK) return s;
  return check_launch();
}

tc_status tc_reassemble(const tc_params* p, int32_t n_sys, int32_t n_text, const void* Hs,
                        const void* Xo, const int32_t* kept_idx, void* Ho, int32_t* pos,
                        void* stream) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (n_sys < 0 || n_text < 0) return TC_ERR_INVALID_ARG;
  if (!Xo || !kept_idx || !Ho || !pos || misaligned(Xo) || misaligned(Ho)) return TC_ERR_INVALID_ARG;
  if ((n_sys > 0 || n_text > 0) && (!Hs || misaligned(Hs))) return TC_ERR_INVALID_ARG;
  launch_reassemble(D, n_sys, n_text, Hs, Xo, kept_idx, Ho, pos, (cudaStream_t)stream);
  return check_launch();
}

tc_status tc_probe_workspace_bytes(const tc_params* p, int32_t n_sys, int32_t n_text, size_t* bytes) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (!bytes || n_sys < 0 || n_text < 0) return TC_ERR_INVALID_ARG;
  *bytes = probe_workspace_bytes(D.B, D.H, n_sys + D.N + n_text, D.dh);
  return TC_OK;
}

tc_status tc_probe(const tc_params* p, int32_t n_sys, int32_t n_text, int32_t probe_start,
                   const void* Q, const void* K, const void* V, void* O, void* A,
                   int32_t* img_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  tc_status s = make_dims(p, &D);
  if (s != TC_OK) return s;
  if (n_sys < 0 || n_text < 0) return TC_ERR_INVALID_ARG;
  const int L = n_sys + D.N + n_text;
  if (!Q || !K || !img_status || (!O && !A) || (O && (!V || !ws))) return TC_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || (V && misaligned(V)) || (O && misaligned(O)) ||
      (A && misaligned(A)) || (ws && misaligned(ws)))
    return TC_ERR_INVALID_ARG;
  if (A && (probe_start < 0 || probe_start + D.T > L)) return TC_ERR_INVALID_ARG;
  if (D.esz != 2 || D.dh != 128 || D.d != D.H * D.dh) return TC_ERR_UNSUPPORTED;
  if (O && ws_bytes < probe_workspace_bytes(D.B, D.H, L, D.dh)) return TC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  fill_i32(img_status, D.B, 0, st);
  s = launch_probe(D.B, D.H, D.dh, L, n_sys, D.N, probe_start, D.T, Q, K, V, O, A, ws, img_status, st,
                   D.bf16 ? 1 : 0);
  if (s != TC_OK) return s;
  return check_launch();
}

tc_status tc_rope_tables(const int32_t* pos, int64_t n_rows, int32_t head_dim, float base,
                         float* cos_out, float* sin_out, void* stream) {
  if (!pos || !cos_out || !sin_out) return TC_ERR_INVALID_ARG;
  if (n_rows < 1 || n_rows > 0x7fffffffLL || head_dim < 2 || (head_dim & 1) || !(base > 1.f))
    return TC_ERR_INVALID_ARG;
  launch_rope_tables(pos, n_rows, head_dim, (double)base, cos_out, sin_out, (cudaStream_t)stream);
  return check_launch();
}

const char* tc_status_string(int32_t status) {
  switch (status) {
    case TC_OK: return "ok";
    case TC_ERR_INVALID_ARG: return "invalid argument";
    case TC_ERR_UNSUPPORTED: return "unsupported shape";
    case TC_ERR_WORKSPACE: return "workspace too small";
    case TC_ERR_NOT_CONVERGED: return "eigen-solver did not converge within max_sweeps";
    case TC_ERR_CUDA: return "CUDA runtime error";
    case TC_ERR_RANK_CAP: return "numerical rank reached rank_cap";
    case TC_ERR_BREAKDOWN: return "Cholesky breakdown";
    case TC_ERR_SCRATCH_LIMIT: return "request exceeds the built-in scratch of tc_attn_score_noalloc";
    default: return "unknown status";
  }
}

int32_t tc_version(void) { return 100; }

tc_status tc_test_fail_tensor_maps(int32_t on) {
  tc::g_refuse_encode.store(on ? 1 : 0);
  return TC_OK;
}

tc_status tc_set_groups(int32_t groups) {
  if (groups < 1 || groups > tc::kMaxGroups) return TC_ERR_INVALID_ARG;
  tc::g_n_groups.store(groups);
  return TC_OK;
}

int32_t tc_profile_begin(void) {
  std::lock_guard<std::mutex> lk(tc::g_prof.mu);
  tc::g_prof.used = 0;
  tc::g_prof.on = true;
  return TC_OK;
}

int32_t tc_profile_end(double* ms, int64_t* launches, int32_t n) {
  std::lock_guard<std::mutex> lk(tc::g_prof.mu);
  tc::g_prof.on = false;
  if (!ms || !launches || n < (int)tc::KC_COUNT) return TC_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    ms[i] = 0.0;
    launches[i] = 0;
  }
  for (size_t s = 0; s < tc::g_prof.used; ++s) {
    if (cudaEventSynchronize(tc::g_prof.ev[2 * s + 1]) != cudaSuccess) return TC_ERR_CUDA;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, tc::g_prof.ev[2 * s], tc::g_prof.ev[2 * s + 1]) != cudaSuccess)
      return TC_ERR_CUDA;
    ms[tc::g_prof.cls[s]] += t;
    launches[tc::g_prof.cls[s]] += tc::g_prof.launches_at_close[s] - tc::g_prof.launches_at_open[s];
  }
  tc::g_prof.used = 0;
  return TC_OK;
}

const char* tc_kernel_class_name(int32_t cls) {
  static const char* names[] = {"fill", "attn_colsum", "gram", "sketch", "gemm_f32_YRinv", "chol_inv",
                                "eig", "ics", "combine", "prune", "match", "merge_select",
                                "compact", "gemm_f32_GQ", "gemm_f32_YtY"};
  return (cls >= 0 && cls < (int)tc::KC_COUNT) ? names[cls] : "?";
}

int64_t tc_launch_count(void) { return (int64_t)tc::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
