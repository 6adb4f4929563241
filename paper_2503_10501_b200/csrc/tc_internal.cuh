// Internal declarations shared by the translation units of libtokencarve.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "tokencarve.h"

#include <atomic>

namespace tc {

// test hook (tc_test_fail_tensor_maps): while set, every tensor-map encode is refused, which is
// how a launcher's refusal after the group streams were forked is exercised without a GPU fault
inline std::atomic<int> g_refuse_encode{0};


// Counts of Sec. 3.3.1 / Eq. 3-9 plus everything the launchers derive from tc_params.
struct Dims {
  int B, N, d, H, dh, T;
  int keep, M, P, nA, nB;
  int k;          // dimension of the decomposed subspace: rank_cap, or N for the full solve
  bool full;      // rank_cap == 0
  bool tcp;       // the subspace solve runs its products on the tensor cores (split panels)
  int esz;        // bytes per element of O, A, X, K, V
  bool f16;       // float16 storage
  bool bf16;      // bfloat16 storage (neither: float32)
  int sim_src;    // Eq. 3-10 features: 0 rows of O (the paper), 1 rows of X, 2 head-mean of K
  bool wmerge;    // merge with the IPGS scores as weights instead of the plain mean
  int chunks;     // row chunks of the attention column-mean
  int max_sweeps;
  float lambda, rank_tol;
  int score_norm;
};

tc_status make_dims(const tc_params* p, Dims* out);

// Offsets (bytes) of every scratch array inside the caller's workspace.
struct Plan {
  size_t s_part;   // [B, chunks, N] f32   partial column sums of A
  size_t S, C, E;  // [B, N] f32 each
  size_t sigma;    // [B, k] f32 (unsorted eigenvalue norms theta)
  size_t G;        // [B, N, N] f32
  size_t Y0, Y1, Y2;  // [B, N, k] f32 each (subspace solve only)
  size_t Sm, Rinv, Hm;  // [B, k, k] f32 each (subspace solve only; Sm, Hm: tn_parts(k) of them)
  size_t W, ZT;    // [B, k, k] f32: Jacobi work matrix and accumulated rotations (column-major)
  size_t setA, setB, best_val, best_dst, msrc, mdst, kept;  // int32 / f32 lists
  size_t rank;     // [B] int32
  size_t flags;    // [B] int32 device status scratch
  size_t Kmean;    // [B, N, dh] f32: head-mean keys (sim_src == 2 only)
  // tensor-core subspace solve (Dims::tcp)
  size_t PA, PB;   // two sets of tall panels: [B][N][k] row-major and, panel_T_off bytes
                   // further on, [B][k][N] transposed
  size_t panel_T_off;
  size_t Sk, Hk;   // [B][k][k] f32: Y^T Y (later the eigenvectors) and the projected matrix
  size_t Es;       // [B][4][k][k] f32 scratch of the tridiagonal solver
  size_t total;
};

Plan make_plan(const Dims& D);

// value rounded to the nearest TF32 (low 13 mantissa bits zero)
__device__ __forceinline__ float tf32_round(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}

// Number of parts per image in which the k x k products of the subspace solve are stored
// (partial sums over chunks of the long dimension, added up by the kernel that reads them).
int tn_parts(int k);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Runs `...` with T bound to the storage type of the call.
#define TC_WITH_STORAGE_TYPE(D, ...)      \
  do {                                    \
    if ((D).bf16) {                       \
      using T = __nv_bfloat16;            \
      __VA_ARGS__                         \
    } else if ((D).f16) {                 \
      using T = __half;                   \
      __VA_ARGS__                         \
    } else {                              \
      using T = float;                    \
      __VA_ARGS__                         \
    }                                     \
  } while (0)

// Running count of kernels this library has launched (host side, all streams).
void note_launch(int n = 1);

// Kernel classes for the optional event profile (tc_profile_begin / tc_profile_end).
enum KernelClass {
  KC_FILL = 0, KC_ATTN, KC_GRAM, KC_SKETCH, KC_GEMM, KC_CHOL, KC_JACOBI, KC_ICS, KC_COMBINE,
  KC_PRUNE, KC_MATCH, KC_MSEL, KC_COMPACT, KC_GEMM_GQ, KC_GEMM_TN, KC_COUNT
};
// While a profile is open, brackets the launches made in its lifetime with two CUDA events
// on `st`; otherwise does nothing.
struct Scope {
  int slot;
  cudaStream_t st;
  Scope(int cls, cudaStream_t st);
  ~Scope();
};

// ---- launchers (each only enqueues on `st`) ---------------------------------------------
// Eq. 3-7: column means of A over heads and query rows.
void launch_attn_colsum(const Dims& D, const void* A, float* s_part, cudaStream_t st);
// Eq. 3-8 (+ the 1/(H T) of Eq. 3-7): S and E from the partial sums and C.
void launch_combine(const Dims& D, const float* s_part, const float* C, float* S, float* E,
                    cudaStream_t st);
// Stage I prune + Eq. 3-9 split.
void launch_prune(const Dims& D, const float* E, int32_t* setA, int32_t* setB, cudaStream_t st);
// Eq. 3-10 best match per Set-B token, from the Gram matrix or from the rows of O.
// (status [B]: receives TC_ERR_INVALID_ARG for an image whose lists hold a token number outside
// [0, N); such an entry is skipped, never used as an address.  The same for the launchers below.)
void launch_match_gram(const Dims& D, const float* G, const int32_t* setA, const int32_t* setB,
                       float* best_val, int32_t* best_dst, int32_t* status, cudaStream_t st);
void launch_match_rows(const Dims& D, const void* O, const int32_t* setA, const int32_t* setB,
                       float* best_val, int32_t* best_dst, int32_t* status, cudaStream_t st);
// top-M of the best similarities, merge lists, kept list.
void launch_merge_select(const Dims& D, const int32_t* setA, const int32_t* setB,
                         const float* best_val, const int32_t* best_dst, int32_t* msrc,
                         int32_t* mdst, int32_t* kept, int32_t* status, cudaStream_t st);
// merge + gather of X, K, V.
// E: the per-token weights [B, N] of the score-weighted merge, or null for the plain mean.
void launch_compact(const Dims& D, const void* X, const void* K, const void* V,
                    const int32_t* kept, const int32_t* msrc, const int32_t* mdst, void* Xo,
                    void* Ko, void* Vo, const float* E, int32_t* status, cudaStream_t st);
// Km [B, N, dh] float32 = mean over the heads of K [B, H, N, dh].
void launch_mean_heads(const Dims& D, const void* K, float* Km, cudaStream_t st);
// launch_match_rows on float32 features F [B, N, f] whatever the storage type of the call.
void launch_match_rows_f32(const Dims& D, const float* F, int f, const int32_t* setA,
                           const int32_t* setB, float* best_val, int32_t* best_dst,
                           int32_t* status, cudaStream_t st);

// Sec. 3.2: rows idx[b][0..n_sub) of O gathered into Os [B, n_sub, d] (D describes O).
void launch_gather_rows(const Dims& D, int n_sub, const void* O, const int32_t* idx, void* Os,
                        int32_t* status, cudaStream_t st);
void fill_i32(int32_t* p, int n, int v, cudaStream_t st);
// Sec. 3.1 / Conclusion: [system, compacted visual, prompt] rows and their original positions.
void launch_reassemble(const Dims& D, int n_sys, int n_text, const void* Hs, const void* Xo,
                       const int32_t* kept, void* Ho, int32_t* pos, cudaStream_t st);

// Conclusion: rotary tables cos / sin [rows][head_dim / 2] of the given position IDs.
void launch_rope_tables(const int32_t* pos, long long rows, int head_dim, double base, float* cosv,
                        float* sinv, cudaStream_t st);

// Layer-2 probe (Eq. 3-1 / 3-2): visual rows of the attention output and the probe rows'
// attention to the visual tokens, from Q, K, V [B, H, L, dh] (16-bit storage, dh = 128).
size_t probe_workspace_bytes(int B, int H, int L, int dh);
tc_status launch_probe(int B, int H, int dh, int L, int n_sys, int n_vis, int probe_start, int n_probe,
                       const void* Q, const void* K, const void* V, void* O, void* A, void* ws,
                       int32_t* status, cudaStream_t st, int bf);

// G = O O^T (float32 out).
tc_status launch_gram(const Dims& D, const void* O, float* G, int32_t* status, cudaStream_t st);

// C [batch][M][NN] = A B^T on the tensor cores, float32-accurate (A [batch][M][K],
// B [batch][NN][K]); C and / or its transpose CT [batch][NN][M] are written (either may be null).
bool gemm_f32x3_supported(int M, int NN, int K);
tc_status launch_gemm_f32x3(const float* A, const float* B, int M, int NN, int K, int batch,
                            float* C, float* CT, int32_t* status, cudaStream_t st, int cls);

// Eigen-decomposition of G and Eq. 3-6:  C, theta (unsorted), then sorted sigma / rank.
// g_ready: optional event after which G is complete when it is built on another stream (the
// subspace solve waits for it in front of its first product with G).
// full_scratch: optional 4 * B * N * N floats; with it a full solve (rank_cap = 0) of a matrix
// that fits in shared memory goes through the tridiagonal solver instead of Jacobi sweeps.
tc_status launch_ics(const Dims& D, const Plan& P, char* ws, int b0, const void* O, float* C_out,
                     float* sigma_out, int32_t* rank_out, int32_t* img_status, cudaStream_t st,
                     float* full_scratch = nullptr, cudaEvent_t g_ready = nullptr);

}  // namespace tc
